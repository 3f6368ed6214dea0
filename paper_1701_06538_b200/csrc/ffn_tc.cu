// Expert feed-forward networks on the 5th-generation tensor cores (Section 3.2, Appendix C):
// variable-size grouped GEMMs, bf16 operands, fp32 accumulation in tensor memory.
//
// One persistent kernel template, one CTA per SM, 128 x 256 output tiles, K blocks of 64:
//   warp 0      TMA producer: one bulk tensor copy per operand per stage into 128-byte-swizzled
//               shared memory, completion counted on an mbarrier (4 stages)
//   warp 1      MMA issuer: tcgen05.mma (cta_group::1, kind::f16, M 128, N 256, K 16), accumulator
//               in TMEM, double buffered (2 x 256 columns) so the epilogue of one tile overlaps
//               the main loop of the next; tcgen05.commit releases the stage / publishes the tile
//   warps 2-9   epilogue: tcgen05.ld (32 lanes x 32 columns per instruction), bias / ReLU / ReLU
//               mask, round to bf16, 64-byte row stores with a row guard for ragged segments
//
// Three operand arrangements (KIND):
//   ROW_BMN  rows x K activations (K-major A) times a per-expert [K, N] weight (N contiguous,
//            "MN-major" B): forward GEMMs  hid = relu(xs.W1 + b1),  ys = hid.W2 + b2
//   ROW_BK   same A, per-expert weight read transposed ([N, K], K contiguous, K-major B):
//            dz = (dys.W2^T) * [hid > 0],  dxs = dz.W1^T
//   WGRAD    contraction over the rows of a segment, both operands MN-major:
//            dW2 = hid^T.dys,  dW1 = xs^T.dz. The last K block of a segment is ragged: the rows
//            past the segment end are zeroed in shared memory in both operands.
// Weights are addressed through one tensor map with the expert as a coordinate, segment bounds
// are read on the device: no per-expert descriptors and no host synchronisation.
//
// Every wait on an mbarrier is bounded (2 s of %globaltimer); on expiry the CTA records
// MOE_ERR_TIMEOUT in the workspace status word, stops issuing work, drains and frees its TMEM.
#include <cuda.h>
#include <stdlib.h>
#include <string.h>

#include "moe_internal.cuh"

namespace moe {

namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;  // 16 KiB
constexpr int B_BYTES = BN * BK * 2;  // 32 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int EPI_STAGE_BYTES = 8 * 4096;  // per epilogue warp: a 32 x 128 B slab for float output
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/ + EPI_STAGE_BYTES;
constexpr int TMEM_COLS = 512;
constexpr int NTHREADS = 320;   // TMA warp, MMA warp, 8 epilogue warps
constexpr int NTHREADS2 = 384;  // two-CTA kernel: + one warp that fixes the ragged K tail of the wgrad ahead of the MMAs, + the tile scheduler warp
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;

enum Kind { ROW_BMN = 0, ROW_BK = 1, WGRAD = 2 };

constexpr int MAX_TERMS = 8;

struct GemmParams {
    const int32_t *offsets;      // [nseg + 1] segment bounds (rows); nullptr = uniform segments
    const int32_t *tile_prefix;  // ROW_* with offsets: [nseg + 1] prefix of the M tiles
    const int4 *tile_info;       // ROW_* with offsets: per M tile {segment or -1, first row, segment end, 0}
    // set by the launchers: N tiles per row of tiles, WGRAD tiles per segment, number of tile ids, K blocks of a ROW tile
    int32_t tiles_n, per_e, total_tiles, kblocks_row;
    int32_t nseg;
    int32_t M;  // WGRAD: rows of the per-segment output; ROW_*: unused
    int32_t N;  // output columns
    int32_t K;  // ROW_*: contraction length of one term; WGRAD: unused (segment rows)
    bf16 *out;  // ROW_*: [R, N]; WGRAD: [nseg, M, N]
    float *out_f32;    // if set, results are written here as float instead of `out`
    const bf16 *bias;  // [nseg, N] or nullptr
    const bf16 *mask;  // [R, N] or nullptr: result kept where mask > 0
    // the same mask as one bit per element, [R, N / 32] words (bit j of word c: column 32 c + j): bits_out is written by
    // the GEMM whose output the mask is taken of (bit = stored value > 0), bits_in is applied like `mask`
    uint32_t *bits_out;
    const uint32_t *bits_in;
    // ROW_* with bf16 output: if set, column sums of the stored values over each epilogue warp's 32 rows,
    // [32-row block][N] floats; block = (global M tile * CTAs per tile + CTA rank) * 4 + row quarter
    float *colsum_part;
    int32_t tma_out;  // two-CTA ROW_*: full 32-row pieces leave through shared memory and bulk tensor stores
    int32_t relu;
    int32_t *status;
    // uniform segments (offsets == nullptr): ROW_*: one segment of R rows. WGRAD: segment s covers
    // rows [c * rows_per_seg, min(R, (c+1) * rows_per_seg)) with c = s % segs_per_term, and reads the
    // B columns shifted by (s / segs_per_term) * b_term_chunks chunks of 64 (split-precision terms).
    int64_t R;
    int32_t rows_per_seg, segs_per_term, b_term_chunks;
    int32_t segs_term0, rows_per_seg0;  // if segs_term0 > 0: term 0 is cut into that many ranges of rows_per_seg0
    int32_t interleave;                 // uniform WGRAD: number of terms whose tiles alternate in the id order (0: none)
    int32_t sub_kb0, sub_kb;            // ACC kernel: K blocks per separately accumulated sub-block, term 0 / other terms
    int32_t off_mod;                    // WGRAD with offsets: see tile_fetch
    // ROW_*: the contraction is the concatenation of nterms pieces of length K; piece i reads A
    // columns a_term_col[i] + [0, K) and B columns b_term_col[i] + [0, K)
    int32_t nterms;
    int32_t a_term_col[MAX_TERMS], b_term_col[MAX_TERMS];
    // two-CTA kernels over ragged segments: tiles are handed out at run time (see PairTiles). sched_counter = next tile
    // id; sched_table[id / sched_group] = {segment, first row, end row, 0} (segment -1: no more tiles). WGRAD: the
    // segments in descending size, sched_group = tiles per segment; ROW_*: tile_info, sched_group = N tiles per M tile
    const int4 *sched_table;
    int32_t *sched_counter;
    int32_t sched_group;
    int32_t trace;  // diagnostics build only: this launch records the tile trace
};

// Diagnostics build (-DMOE_TILE_TRACE): the first CTA records, per tile, when each warp role started, finished and how
// long it waited; read back with moe_debug_tile_trace. Compiled out otherwise.
#ifdef MOE_TILE_TRACE
__device__ long long g_tile_trace[3][256][6];
#define TILE_TRACE_SET(role, tile, field, val) do { if (p.trace && blockIdx.x == 0 && (tile) < 256) g_tile_trace[role][tile][field] = (val); } while (0)

#define TILE_CLOCK() clock64()
static int g_trace_launch_no = 0;
#else
#define TILE_TRACE_SET(role, tile, field, val) do {} while (0)
#define TILE_CLOCK() 0ll
#endif

// ------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// same, with cluster-scope acquire (the arrival comes from the other CTA of the pair)
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait. Returns false (and raises the CTA's abort flag + the status word) on expiry.
__device__ __forceinline__ bool mbar_wait_limit(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *status,
                                                unsigned long long limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_ns() - t0 > limit_ns) {
            *abort_flag = 1;
            atomicExch(status, (int32_t)MOE_ERR_TIMEOUT);
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *status) {
    return mbar_wait_limit(bar, parity, abort_flag, status, WAIT_LIMIT_NS);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tm, uint32_t bar, int c0, int c1,
                                            int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *tm, uint32_t bar, int c0, int c1,
                                            int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], "
        "[%2];" ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}

// bulk tensor store of a [32 rows][64 columns] box from 128-byte-swizzled shared memory
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *tm, uint32_t src, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(tm), "r"(src), "r"(c0),
                 "r"(c1)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// 256-bit store (sm_100): a whole 32-byte sector per instruction
__device__ __forceinline__ void st_global_32B(uint4 *dst, const uint4 &a, const uint4 &b) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(a.x), "r"(a.y), "r"(a.z),
                 "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w)
                 : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptors (128-byte swizzle, descriptor version 1 at bit 46).
// K-major: rows of 64 bf16 (128 B); 8-row groups 1024 B apart (stride byte offset).
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t addr) {
    return (uint64_t)((addr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// MN-major: 64 contiguous MN elements (128 B) per K row; 8 K rows per 1024-B atom (stride byte
// offset); the next 64 MN elements start BK * 128 B further (leading byte offset).
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr) {
    return (uint64_t)((addr & 0x3FFFF) >> 4) | ((uint64_t)((BK * 128) >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor: D fp32, A/B bf16, majors, N >> 3 at bit 17, M >> 4 at bit 24.
__host__ __device__ constexpr uint32_t make_idesc(int a_mn, int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

// Column sums over the 32 rows a warp holds (one row per lane, 32 columns per lane): returns in lane l
// the sum of column l. Butterfly: each step a lane keeps one half of its columns and sends the other.
__device__ __forceinline__ float warp_column_sums(float (&a)[32], int lane) {
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        const bool up = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < s; ++i) {
            const float keep = up ? a[i + s] : a[i];
            const float send = up ? a[i] : a[i + s];
            a[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
        }
    }
    return a[0];
}

// Epilogue arithmetic of one thread's 32 accumulator columns: bias, ReLU, ReLU mask, rounding to bf16. The three
// options are template parameters so that the loop body has no branches (with run-time flags every element pair became
// its own basic block and the chain add -> max -> convert ran serially, 16 times).
template <bool BIAS, bool RELU, bool MASK, bool BITS = false>
__device__ __forceinline__ void pack32_mode(const uint32_t (&v)[32], const uint4 (&bias_raw)[4], const uint4 (&mask_raw)[4],
                                            uint4 (&packed)[4], uint32_t keep_word = 0u) {
    const uint32_t *bw = reinterpret_cast<const uint32_t *>(bias_raw);
    const uint32_t *mw = reinterpret_cast<const uint32_t *>(mask_raw);
    uint32_t *out = reinterpret_cast<uint32_t *>(packed);
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        float x0 = __uint_as_float(v[2 * j]), x1 = __uint_as_float(v[2 * j + 1]);
        if (BIAS) { x0 += __uint_as_float(bw[j] << 16); x1 += __uint_as_float(bw[j] & 0xffff0000u); }
        if (RELU) { x0 = fmaxf(x0, 0.0f); x1 = fmaxf(x1, 0.0f); }
        if (MASK) {
            if (!(__uint_as_float(mw[j] << 16) > 0.0f)) x0 = 0.0f;
            if (!(__uint_as_float(mw[j] & 0xffff0000u) > 0.0f)) x1 = 0.0f;
        }
        if (BITS) {
            if (!((keep_word >> (2 * j)) & 1u)) x0 = 0.0f;
            if (!((keep_word >> (2 * j + 1)) & 1u)) x1 = 0.0f;
        }
        const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
        out[j] = *reinterpret_cast<const uint32_t *>(&h);
    }
}
// one bit per packed value: set where the stored bf16 value is greater than zero
__device__ __forceinline__ uint32_t positive_bits(const uint4 (&packed)[4]) {
    const uint32_t *pw = reinterpret_cast<const uint32_t *>(packed);
    uint32_t word = 0u;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const uint32_t lo = pw[j] & 0xffffu, hi = pw[j] >> 16;
        word |= (uint32_t)(lo != 0u && !(lo & 0x8000u)) << (2 * j);
        word |= (uint32_t)(hi != 0u && !(hi & 0x8000u)) << (2 * j + 1);
    }
    return word;
}
// mode: bit 0 bias, bit 1 ReLU, bit 2 mask, bit 3 mask as bits (the combinations the layer uses are specialised)
__device__ __forceinline__ void pack32(int mode, const uint32_t (&v)[32], const uint4 (&bias_raw)[4],
                                       const uint4 (&mask_raw)[4], uint4 (&packed)[4], uint32_t keep_word = 0u) {
    if (mode & 8) {
        pack32_mode<false, false, false, true>(v, bias_raw, mask_raw, packed, keep_word);
        return;
    }
    switch (mode) {
        case 0: pack32_mode<false, false, false>(v, bias_raw, mask_raw, packed); break;
        case 1: pack32_mode<true, false, false>(v, bias_raw, mask_raw, packed); break;
        case 3: pack32_mode<true, true, false>(v, bias_raw, mask_raw, packed); break;
        case 4: pack32_mode<false, false, true>(v, bias_raw, mask_raw, packed); break;
        case 2: pack32_mode<false, true, false>(v, bias_raw, mask_raw, packed); break;
        case 5: pack32_mode<true, false, true>(v, bias_raw, mask_raw, packed); break;
        case 6: pack32_mode<false, true, true>(v, bias_raw, mask_raw, packed); break;
        default: pack32_mode<true, true, true>(v, bias_raw, mask_raw, packed); break;
    }
}

// The bias values of one warp's 128 output columns are fetched before the warp waits for its accumulator (the load
// latency used to sit between the tensor-memory load and the arithmetic of every 32-column piece): lane l < 16 holds
// the 16-byte piece l; piece 4 * ci + q, q = 0..3, of the ci-th 32-column piece is handed to every lane by shuffles.
__device__ __forceinline__ uint4 bias_slice_load(const bf16 *bias, int64_t row_off, int32_t col_first, int32_t N, int lane) {
    uint4 v = make_uint4(0, 0, 0, 0);
    if (bias && lane < 16 && col_first + lane * 8 < N) v = *reinterpret_cast<const uint4 *>(bias + row_off + col_first + lane * 8);
    return v;
}
__device__ __forceinline__ void bias_slice_piece(const uint4 &mine, int ci, uint4 (&out)[4]) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        out[q].x = __shfl_sync(0xffffffffu, mine.x, 4 * ci + q);
        out[q].y = __shfl_sync(0xffffffffu, mine.y, 4 * ci + q);
        out[q].z = __shfl_sync(0xffffffffu, mine.z, 4 * ci + q);
        out[q].w = __shfl_sync(0xffffffffu, mine.w, 4 * ci + q);
    }
}

struct Tile {
    int32_t e;        // expert / segment
    int32_t row0;     // ROW_*: first sorted row; WGRAD: first row of the segment
    int32_t row_end;  // end of the segment
    int32_t m0;       // WGRAD: first output row of the tile
    int32_t n0;       // first output column
    int32_t kblocks;  // number of K blocks
    int32_t b_chunk;  // WGRAD: first 64-column chunk of B
    int32_t mt;       // ROW_*: index of the M tile over all segments
};

// Tile ids are handed out round-robin. What a tile needs from global memory (its segment's bounds) is
// fetched one tile ahead (tile_fetch) and only turned into a Tile (tile_decode) when the tile starts, so
// the load latency never sits between two tiles. ROW_* with ragged segments read one 16-byte record per
// M tile from a table built by tile_table_kernel; WGRAD reads the two segment bounds.
template <int KIND>
__device__ __forceinline__ int4 tile_fetch(const GemmParams &p, int32_t id) {
    if (!p.offsets || id >= p.total_tiles) return make_int4(-1, 0, 0, 0);
    if (KIND == WGRAD) {
        const int32_t e = id / p.per_e;
        const int32_t seg = p.off_mod > 0 ? e % p.off_mod : e;  // with off_mod: segment s reads the rows of group s % off_mod
        return make_int4(e, p.offsets[seg], p.offsets[seg + 1], 0);
    }
    return p.tile_info[id / p.tiles_n];
}

template <int KIND, int TM>
__device__ __forceinline__ bool tile_decode(const GemmParams &p, int32_t id, const int4 &raw, Tile &t) {
    if (id >= p.total_tiles) return false;
    if (KIND == WGRAD) {
        int32_t e = id / p.per_e;
        const int32_t rem = id - e * p.per_e;
        // uniform ranges, interleaved terms: consecutive ids walk the terms of one row range (its rows stay in L2 for all
        // of them) while the segment index stays term-major
        if (p.interleave > 1) e = (e % p.interleave) * p.segs_per_term + e / p.interleave;
        const int32_t tm = rem / p.tiles_n;
        t.e = e;
        t.mt = 0;
        t.m0 = tm * TM;
        t.n0 = (rem - tm * p.tiles_n) * BN;
        t.b_chunk = t.n0 / 64;
        if (p.offsets) {
            t.row0 = raw.y;
            t.row_end = raw.z;
            if (p.off_mod > 0) t.b_chunk += (e / p.off_mod) * p.b_term_chunks;  // B term s / off_mod
        } else {
            int64_t c, rps;
            int32_t term;
            if (e < p.segs_term0) {  // term 0 may use its own (shorter) row ranges
                c = e; rps = p.rows_per_seg0; term = 0;
            } else {
                const int32_t e2 = e - p.segs_term0;
                c = e2 % p.segs_per_term; rps = p.rows_per_seg;
                term = e2 / p.segs_per_term + (p.segs_term0 > 0 ? 1 : 0);
            }
            t.row0 = (int32_t)(c * rps);
            t.row_end = (int32_t)(((c + 1) * rps < p.R) ? (c + 1) * rps : p.R);
            if (t.row_end < t.row0) t.row_end = t.row0;
            t.b_chunk += term * p.b_term_chunks;
        }
        t.kblocks = (t.row_end - t.row0 + BK - 1) / BK;
        return true;
    } else {
        const int32_t mt = id / p.tiles_n;
        t.mt = mt;
        t.m0 = 0;
        t.b_chunk = 0;
        t.kblocks = p.kblocks_row;
        t.n0 = (id - mt * p.tiles_n) * BN;
        if (!p.offsets) {  // one segment of R rows; total_tiles is exact
            t.e = 0;
            t.row0 = mt * TM;
            t.row_end = (int32_t)p.R;
            return true;
        }
        if (raw.x < 0) return false;  // past the last M tile
        MOE_BOUNDS_NOTE(raw.x < p.nseg && raw.y >= 0 && raw.y <= raw.z && (int64_t)raw.z <= p.R);
        t.e = raw.x;
        t.row0 = raw.y;
        t.row_end = raw.z;
        return true;
    }
}

template <int KIND, int TM> struct TileIter {
    const GemmParams &p;
    int32_t id, stride;
    int4 raw;
    __device__ __forceinline__ TileIter(const GemmParams &p_, int32_t first, int32_t stride_)
        : p(p_), id(first), stride(stride_) { raw = tile_fetch<KIND>(p, id); }
    // the current tile; starts the fetch for the following one
    __device__ __forceinline__ bool next(Tile &t) {
        if (!tile_decode<KIND, TM>(p, id, raw, t)) return false;
        id += stride;
        raw = tile_fetch<KIND>(p, id);
        return true;
    }
};

// ACC (WGRAD with float output over long uniform row ranges, the gate backward): the contraction of a tile is cut
// into sub-blocks of p.sub_kb0 / p.sub_kb K blocks (first term / other terms). Each sub-block is accumulated in TMEM on
// its own (an fp32 tensor-core accumulator truncates, and a long run of same-sign terms loses low bits: 128 rows keep
// that below 1e-5), handed to the epilogue like a tile, and added there, with rounding to nearest, to running sums in
// shared memory (32 rows x 128 columns of floats per warp, 16-byte units swizzled by row); the sums go to global memory
// once per tile. Two stages of operands make room for the 128 KiB of sums.
template <int KIND, bool ACC = false>
__global__ void __launch_bounds__(NTHREADS, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // 1024-B aligned for the 128-B swizzle
    uint8_t *smem = smem_raw + (base - smem_u32(smem_raw));
    constexpr int NST = ACC ? 2 : STAGES;
    const uint32_t bars = base + NST * STAGE_BYTES;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (NST + s); };
    auto tfull_bar = [&](int a) { return bars + 8u * (2 * NST + a); };
    auto tempty_bar = [&](int a) { return bars + 8u * (2 * NST + 2 + a); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + NST * STAGE_BYTES + 8 * (2 * NST + 4));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + NST * STAGE_BYTES + 8 * (2 * NST + 4) + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)),
                     "r"((uint32_t)TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            TileIter<KIND, BM> it(p, (int32_t)blockIdx.x, (int32_t)gridDim.x);
            Tile t;
            while (ok && it.next(t)) {
                int term = 0, kk = 0;  // ROW_*: piece of the contraction and column inside it
                for (int kb = 0; kb < t.kblocks && ok; ++kb) {
                    ok = mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status);
                    if (!ok) break;
                    const uint32_t a_dst = base + s * STAGE_BYTES, b_dst = a_dst + A_BYTES;
                    mbar_expect_tx(full_bar(s), STAGE_BYTES);
                    if (KIND == WGRAD) {
                        const int r = t.row0 + kb * BK;
                        tma_load_3d(a_dst, &tmA, full_bar(s), 0, r, t.m0 / 64);
                        tma_load_3d(b_dst, &tmB, full_bar(s), 0, r, t.b_chunk);
                    } else {
                        tma_load_2d(a_dst, &tmA, full_bar(s), p.a_term_col[term] + kk, t.row0);
                        if (KIND == ROW_BMN) tma_load_4d(b_dst, &tmB, full_bar(s), 0, p.b_term_col[term] + kk, t.n0 / 64, t.e);
                        else tma_load_3d(b_dst, &tmB, full_bar(s), p.b_term_col[term] + kk, t.n0, t.e);
                        kk += BK;
                        if (kk == p.K) { kk = 0; ++term; }
                    }
                    if (++s == NST) { s = 0; ph ^= 1u; }
                }
            }
            // drain: every copy this thread started must have landed before the CTA may exit
            if (!ok)
                for (int q = 0; q < NST; ++q) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(full_bar(q), 0) && !mbar_try_wait(full_bar(q), 1) &&
                           global_ns() - t0 < WAIT_LIMIT_NS) {}
                }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        constexpr uint32_t idesc = make_idesc(KIND == WGRAD ? 1 : 0, KIND == ROW_BK ? 0 : 1);
        int s = 0, acc = 0;
        uint32_t ph = 0, acc_ph = 0;
        bool ok = true;
        TileIter<KIND, BM> it(p, (int32_t)blockIdx.x, (int32_t)gridDim.x);
        Tile t;
        while (ok && it.next(t)) {
            if (t.kblocks == 0) continue;  // empty segment (WGRAD): the epilogue writes zeros
            const int sub = ACC ? (t.e < p.segs_term0 ? p.sub_kb0 : p.sub_kb) : t.kblocks;  // K blocks per accumulator
            uint32_t d_tmem = tmem_base + acc * BN;
            for (int kb = 0; kb < t.kblocks; ++kb) {
                const int kin = ACC ? kb % sub : kb;  // K block inside the accumulator's sub-block
                if (kin == 0) {
                    ok = mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    d_tmem = tmem_base + acc * BN;
                }
                ok = mbar_wait(full_bar(s), ph, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_src = base + s * STAGE_BYTES, b_src = a_src + A_BYTES;
                int ksteps = BK / 16;  // K steps of 16 rows to issue for this block
                if (KIND == WGRAD && kb == t.kblocks - 1) {
                    const int valid = t.row_end - (t.row0 + kb * BK);  // rows of this block inside the segment
                    if (valid < BK) {
                        // The rows behind the segment's end belong to the next segment. Whole K steps behind it are not
                        // issued at all; in the step that holds the end, K rows [valid, end of the step) are zeroed in A
                        // AND in B (0 x finite = 0 would do for finite data; both keep a non-finite value of the next
                        // segment out of this segment's sums): 128-B lines in all 64-column chunks, the A tile's two
                        // chunks directly followed by the B tile's four.
                        ksteps = (valid + 15) / 16;
                        const int nz = ksteps * 16 - valid;
                        const int lines = nz * ((BM + BN) / 64);
                        for (int u = lane; u < lines * 8; u += 32) {
                            const int line = u >> 3, part = u & 7;
                            const int chunk = line / nz, krow = valid + line % nz;
                            *reinterpret_cast<uint4 *>(smem + s * STAGE_BYTES + chunk * (BK * 128) + krow * 128 + part * 16) =
                                make_uint4(0, 0, 0, 0);
                        }
                        if (nz > 0) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                    }
                }
                if (lane == 0) {
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        if (k >= ksteps) break;
                        uint64_t ad, bd;
                        if (KIND == WGRAD) ad = desc_mnmajor(a_src + k * 16 * 128);
                        else ad = desc_kmajor(a_src + k * 32);
                        if (KIND == ROW_BK) bd = desc_kmajor(b_src + k * 32);
                        else bd = desc_mnmajor(b_src + k * 16 * 128);
                        tc_mma_bf16(d_tmem, ad, bd, idesc, (kin > 0 || k > 0) ? 1u : 0u);
                    }
                    tc_commit(empty_bar(s));  // the stage may be refilled once these MMAs have read it
                }
                __syncwarp();
                if (++s == NST) { s = 0; ph ^= 1u; }
                if (ACC && (kin == sub - 1 || kb == t.kblocks - 1)) {  // sub-block complete
                    if (lane == 0) tc_commit(tfull_bar(acc));
                    __syncwarp();
                    if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
                }
            }
            if (!ACC) {
                if (ok && lane == 0) tc_commit(tfull_bar(acc));  // accumulator complete
                __syncwarp();
                if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..9)
        const int quarter = warp & 3;  // TMEM lanes 32*quarter .. 32*quarter + 31 belong to this warp
        const int pack_mode = p.bits_in ? 8 : (p.bias ? 1 : 0) | (p.relu ? 2 : 0) | (p.mask ? 4 : 0);
        int acc = 0;
        uint32_t acc_ph = 0;
        bool ok = true;
        TileIter<KIND, BM> it(p, (int32_t)blockIdx.x, (int32_t)gridDim.x);
        Tile t;
        while (ok && it.next(t)) {
            const bool have_acc = t.kblocks > 0;
            if (ACC) {
                const int half_a = (warp - 2) >> 2;
                uint8_t *sums = smem + NST * STAGE_BYTES + 256 + (warp - 2) * 16384;  // [32 rows][32 x 16 B], unit ^ row
                const int sub = t.e < p.segs_term0 ? p.sub_kb0 : p.sub_kb;
                const int nsub = (t.kblocks + sub - 1) / sub;
                for (int sb = 0; sb < nsub && ok; ++sb) {
                    ok = mbar_wait(tfull_bar(acc), acc_ph, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int cl = 0; cl < 4; ++cl) {
                        uint32_t v[32];
                        tc_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN + (half_a * 4 + cl) * 32, v);
                        tc_ld_wait();
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            float4 *cell = reinterpret_cast<float4 *>(sums + lane * 512 + ((((cl * 8 + q) ^ lane) & 31) << 4));
                            float4 a = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                                   __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                            if (sb > 0) {
                                const float4 o = *cell;
                                a.x += o.x; a.y += o.y; a.z += o.z; a.w += o.w;
                            }
                            *cell = a;
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty_bar(acc));
                    if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
                }
                if (!ok) break;
                // the warp's 32 x 128 sums to global memory, one 512-byte row segment per instruction
                const int64_t row0 = (int64_t)t.m0 + quarter * 32;
                float *dst = p.out_f32 + (int64_t)t.e * p.M * p.N + row0 * p.N + t.n0 + half_a * 128 + lane * 4;
                if (t.n0 + half_a * 128 + lane * 4 < p.N) {
                    for (int i = 0; i < 32; ++i) {
                        if (row0 + i >= p.M) break;
                        float4 val = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                        if (nsub > 0) val = *reinterpret_cast<const float4 *>(sums + i * 512 + (((lane ^ i) & 31) << 4));
                        *reinterpret_cast<float4 *>(dst + (int64_t)i * p.N) = val;
                    }
                }
                __syncwarp();  // the sums are read before the next tile overwrites them
                continue;
            }
            const int half_w = (warp - 2) >> 2;
            const uint4 bias_mine = bias_slice_load(p.bias, (int64_t)t.e * p.N, t.n0 + half_w * (BN / 2), p.N, lane);
            if (have_acc) {
                ok = mbar_wait(tfull_bar(acc), acc_ph, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
            }
            // Two warps share each quarter of the accumulator's rows and take half of its columns each.
            // A thread owns one row. bf16 results are stored straight from registers (64 B per thread and
            // step); float results (128 B per row and step) go through a swizzled shared-memory slab so that
            // the stores are whole 128-byte row segments: lane l moves piece l % 8 of row 4 * i + l / 8.
            const int half = (warp - 2) >> 2;
            uint8_t *stage_o = smem + STAGES * STAGE_BYTES + 256 + (warp - 2) * 4096;
            int64_t tile_row0;   // first output row of this warp's 32 rows
            int32_t rows_valid;  // how many of them exist
            int64_t out_off = 0;
            if (KIND == WGRAD) {
                out_off = (int64_t)t.e * p.M * p.N;
                tile_row0 = t.m0 + quarter * 32;
                rows_valid = p.M - (int32_t)tile_row0;
            } else {
                tile_row0 = (int64_t)t.row0 + quarter * 32;
                rows_valid = t.row_end - (int32_t)tile_row0;
            }
            const int my_piece = lane & 7, my_sub = lane >> 3;
            const bool row_ok = lane < rows_valid;
            const int64_t out_row = tile_row0 + lane;
            for (int c = half * (BN / 64); c < (half + 1) * (BN / 64); ++c) {
                const int col0 = t.n0 + c * 32;
                if (col0 >= p.N) break;
                uint32_t v[32];
                if (have_acc) {
                    tc_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN + c * 32, v);
                    tc_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                uint4 bias_raw[4];
                if (p.bias) bias_slice_piece(bias_mine, c - half * (BN / 64), bias_raw);  // whole warp: shuffles
                if (p.out_f32) {
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        *reinterpret_cast<uint4 *>(stage_o + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                            make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int row = 4 * i + my_sub;
                        if (row < rows_valid)
                            *reinterpret_cast<uint4 *>(p.out_f32 + out_off + (tile_row0 + row) * p.N + col0 + my_piece * 4) =
                                *reinterpret_cast<const uint4 *>(stage_o + row * 128 + ((my_piece ^ (row & 7)) << 4));
                    }
                    __syncwarp();
                } else if (row_ok || p.colsum_part) {  // with column sums the whole warp takes part (shuffles)
                    uint4 packed[4];
                    uint4 mask_raw[4];
                    if (p.mask && row_ok) {
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            mask_raw[q] = reinterpret_cast<const uint4 *>(p.mask + out_row * p.N + col0)[q];
                    }
                    uint32_t keep_word = 0u;
                    if (p.bits_in && row_ok) keep_word = p.bits_in[out_row * (p.N >> 5) + (col0 >> 5)];
                    pack32(pack_mode, v, bias_raw, mask_raw, packed, keep_word);
                    if (p.bits_out && row_ok) p.bits_out[out_row * (p.N >> 5) + (col0 >> 5)] = positive_bits(packed);
                    if (row_ok) {
                        uint4 *dst = reinterpret_cast<uint4 *>(p.out + out_off + out_row * p.N + col0);
                        st_global_32B(dst, packed[0], packed[1]);  // two full 32-byte sectors per row piece
                        st_global_32B(dst + 2, packed[2], packed[3]);
                    }
                    if (p.colsum_part) {  // sums of the rounded values, rows past the segment end count as 0
                        float a[32];
                        const uint32_t *pw = reinterpret_cast<const uint32_t *>(packed);
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            a[2 * j] = row_ok ? __uint_as_float(pw[j] << 16) : 0.0f;
                            a[2 * j + 1] = row_ok ? __uint_as_float(pw[j] & 0xffff0000u) : 0.0f;
                        }
                        const float sum = warp_column_sums(a, lane);
                        p.colsum_part[(int64_t)(t.mt * 4 + quarter) * p.N + col0 + lane] = sum;
                    }
                }
            }
            if (have_acc) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty_bar(acc));
                if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS)
                     : "memory");
    }
}


// ------------------------------------------------------------------------------------------
// Two-CTA variant for the row GEMMs (ROW_BMN, ROW_BK): a cluster of two CTAs (an SM pair) works on a
// 256 x 256 tile with tcgen05.mma cta_group::2 (M 256). Each CTA stages its own 128 rows of A and its
// own 128 columns of B (32 KiB per stage instead of 48, six stages), the pair's tensor cores exchange
// the B halves, and each CTA keeps the accumulator of its 128 rows in its own TMEM. The even CTA of
// the pair issues the MMAs; the loads of both CTAs count on its "full" barrier; tcgen05.commit
// releases a stage / publishes an accumulator in both CTAs at once; the odd CTA's epilogue warps
// hand their accumulator buffer back with an arrive on the even CTA's barrier.
// ------------------------------------------------------------------------------------------
constexpr int STAGES2 = 6;
constexpr int A2_BYTES = 128 * BK * 2, B2_BYTES = 128 * BK * 2, STAGE2_BYTES = A2_BYTES + B2_BYTES;
constexpr int DATA2_BYTES = STAGES2 * STAGE2_BYTES + EPI_STAGE_BYTES;  // 224 KiB: 6 stages + float staging, or 5 stages + mask tile
constexpr int SMEM2_BYTES = DATA2_BYTES + 1024 + 512;  // + alignment slack, barriers, scheduler ring
constexpr uint32_t PEER_BIT_MASK = 0xFEFFFFFFu;  // clears the CTA-rank bit of a shared::cluster address of the pair

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive on the barrier at this shared-memory offset in the EVEN CTA of the pair
__device__ __forceinline__ void mbar_arrive_leader(uint32_t bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar & PEER_BIT_MASK) : "memory");
}
// The same without release semantics, for handing an accumulator buffer back: the tensor-memory reads are
// complete (tcgen05.wait::ld) and fenced (tcgen05.fence::before_thread_sync) before the arrive, and nothing
// the other side reads was written through memory. A release at cluster scope would wait here for all of this
// thread's earlier global stores (the output rows) to reach L2, several thousand cycles per tile.
__device__ __forceinline__ void mbar_arrive_leader_relaxed(uint32_t bar) {
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar & PEER_BIT_MASK) : "memory");
}
__device__ __forceinline__ void tc_commit2(uint32_t bar) {  // arrives at this offset in both CTAs of the pair
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((uint16_t)3)
        : "memory");
}
__device__ __forceinline__ void tc_mma2_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
// loads of the pair: both CTAs' transaction bytes are counted on the even CTA's barrier
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap *tm, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar & PEER_BIT_MASK), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma2_load_3d(uint32_t dst, const CUtensorMap *tm, uint32_t bar, int c0, int c1,
                                             int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar & PEER_BIT_MASK), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tma2_load_4d(uint32_t dst, const CUtensorMap *tm, uint32_t bar, int c0, int c1,
                                             int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], "
        "[%2];" ::"r"(dst), "l"(tm), "r"(bar & PEER_BIT_MASK), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__host__ __device__ constexpr uint32_t make_idesc2(int a_mn, int b_mn) {  // M 256, N 256
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

// Tile source of the two-CTA kernel. Static mode: ids dealt round-robin to the pairs (TileIter). Dynamic mode (ragged
// segments): a fixed deal leaves pairs idle at the end, because the tiles of a weight-gradient GEMM differ in length by
// the ratio of the largest to the smallest expert, and because SM pairs do not all run at the same speed (distance to
// the L2 slices, the two dies). The scheduler warp of the even CTA draws tile ids from a global counter (WGRAD: in
// descending order of segment size, longest first) and publishes one 16-byte record per tile {segment, first row,
// end row, tile id} in a four-slot ring in the shared memory of BOTH CTAs; every warp role of both CTAs reads the
// same sequence of records. A record with segment -1 ends the sequence. Which pair computes a tile does not change
// the tile's result, so the output stays bit-reproducible.
constexpr int SCHED_SLOTS = 4;
__device__ __forceinline__ uint32_t peer_smem_addr(uint32_t addr, uint32_t cta) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(cta));
    return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t addr, const int4 &v) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster_addr(uint32_t cluster_addr) {  // release at cluster scope
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

template <int KIND> struct PairTiles {
    const GemmParams &p;
    TileIter<KIND, 256> fixed;
    const bool dyn, warp_wide, arrives;
    const uint32_t ring, full0, empty0;
    volatile int *abort_flag;
    int i;
    // warp_wide: all 32 lanes of the warp call next() together; arrives: this thread reports the slot as read
    __device__ __forceinline__ PairTiles(const GemmParams &p_, bool dyn_, int32_t first, int32_t stride, uint32_t ring_,
                                         uint32_t full0_, uint32_t empty0_, volatile int *abort_, bool warp_wide_, bool arrives_)
        : p(p_), fixed(p_, dyn_ ? p_.total_tiles : first, stride), dyn(dyn_), warp_wide(warp_wide_), arrives(arrives_),
          ring(ring_), full0(full0_), empty0(empty0_), abort_flag(abort_), i(0) {}
    __device__ __forceinline__ bool next(Tile &t) {
        if (!dyn) return fixed.next(t);
        const int slot = i & (SCHED_SLOTS - 1);
        const uint32_t par = (uint32_t)(i / SCHED_SLOTS) & 1u;
        if (!mbar_wait(full0 + 8u * slot, par, abort_flag, p.status)) return false;
        mbar_try_wait_cluster(full0 + 8u * slot, par);  // acquire at cluster scope: the record came from the other CTA's thread
        // The slot is overwritten once every reader has reported it read, so a reader's copy has to be in its registers
        // before its report leaves. The report is a relaxed arrive (a release at cluster scope would wait for the thread's
        // earlier output stores, 3 % of a step), which by itself orders nothing: with an ordinary load the assembler was
        // free to fetch the record again later instead of keeping it in registers, and in the register-heaviest epilogue
        // (mask bits + column sums) one warp then now and again worked on the record of four tiles ahead and left its
        // piece of the output unwritten. Hence a volatile load (issued once, where it stands) and an arrive whose address
        // is computed from the loaded words of all lanes (sign bit of the tile id, always 0), which cannot issue before
        // those loads have returned.
        int4 rec;
        asm volatile("ld.volatile.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(rec.x), "=r"(rec.y), "=r"(rec.z), "=r"(rec.w)
                     : "r"(ring + 16u * slot) : "memory");
        uint32_t seen = (uint32_t)rec.w;
        if (warp_wide) seen = __reduce_or_sync(0xffffffffu, seen);
        if (arrives) mbar_arrive_leader_relaxed(empty0 + 8u * slot + ((seen >> 31) << 3));
        ++i;
        if (rec.x < 0) return false;
        MOE_BOUNDS_NOTE(rec.x < p.nseg && rec.y >= 0 && rec.y <= rec.z && (int64_t)rec.z <= p.R);
        t.e = rec.x; t.row0 = rec.y; t.row_end = rec.z;
        const int32_t grp = rec.w / p.sched_group, rem = rec.w - grp * p.sched_group;  // rec.w: the tile id
        if (KIND == WGRAD) {
            const int32_t tm = rem / p.tiles_n;
            t.mt = 0;
            t.m0 = tm * 256;
            t.n0 = (rem - tm * p.tiles_n) * BN;
            t.b_chunk = t.n0 / 64;
            t.kblocks = (t.row_end - t.row0 + BK - 1) / BK;
        } else {
            t.mt = grp;
            t.m0 = 0;
            t.b_chunk = 0;
            t.n0 = rem * BN;
            t.kblocks = p.kblocks_row;
        }
        return true;
    }
};

// MASKT: the ReLU mask of the dgrad GEMM is not read row by row from global memory by the epilogue but
// fetched as a 128 x 256 tile by TMA (one stage fewer in exchange for the 64 KiB it occupies).
template <int KIND, bool MASKT>
__global__ void __launch_bounds__(NTHREADS2, 1)
grouped_gemm2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                     const __grid_constant__ CUtensorMap tmM, const __grid_constant__ CUtensorMap tmO,
                     const GemmParams p) {
    // ROW_* with a mask tile: 5 stages and a 64 KiB region of four [128 rows][64 columns] blocks (128-byte swizzle) that
    // holds the ReLU-mask tile and stages the bf16 output for bulk tensor stores; every other kind: 6 stages + 32 KiB of
    // staging (row GEMMs: two such blocks, a warp's two output boxes of a tile pass through the same 4 KiB one after
    // the other; the sixth stage took a seventh off the time the MMA thread waited for operands at 16 K blocks per tile)
    constexpr int NST = (KIND == WGRAD || !MASKT) ? 6 : 5;  // the mask tile needs the 64 KiB region, everything else 32 KiB
    constexpr bool ONE_BOX = KIND != WGRAD && !MASKT;       // row GEMM without a mask tile: one staging box per warp
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + DATA2_BYTES;  // [stages][float staging or mask tile] then the barriers
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (NST + s); };
    auto tfull_bar = [&](int a) { return bars + 8u * (2 * NST + a); };
    auto tempty_bar = [&](int a) { return bars + 8u * (2 * NST + 2 + a); };
    // WGRAD only: afull = this CTA's own tiles of a ragged last K block have landed (the tail rows are zeroed before use);
    // ready (even CTA) = both CTAs' tiles are landed and fixed
    auto afull_bar = [&](int s) { return bars + 8u * (2 * NST + 4 + s); };
    auto ready_bar = [&](int s) { return bars + 8u * (3 * NST + 4 + s); };
    const uint32_t mfull_bar = bars + 8u * 28, mempty_bar = bars + 8u * 29;  // mask tile landed / read by all 8 epilogue warps
    // dynamic tile scheduling (WGRAD): record published / record read by every role of both CTAs (barrier in the even CTA)
    const uint32_t sched_full0 = bars + 256, sched_empty0 = bars + 256 + 8u * SCHED_SLOTS, sched_ring = bars + 384;
    const bool dyn = p.sched_counter != nullptr;
    const uint32_t mask_smem = base + NST * STAGE2_BYTES;                     // 4 blocks of [128 rows][64 columns], 128-B swizzle
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + DATA2_BYTES + 240);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + DATA2_BYTES + 248);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();  // 0: issues the MMAs, owns the full / tempty barriers
    const int64_t cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) {
            mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1);
            mbar_init(afull_bar(s), 1); mbar_init(ready_bar(s), 2);  // ready: both CTAs' tail-fixing warps
        }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 16); }
        mbar_init(mfull_bar, 1); mbar_init(mempty_bar, 8);
        // readers of a scheduler record: producer, 8 epilogue warps (WGRAD: + tail warp) in each CTA, the MMA thread in the even one
        for (int q = 0; q < SCHED_SLOTS; ++q) { mbar_init(sched_full0 + 8u * q, 1); mbar_init(sched_empty0 + 8u * q, KIND == WGRAD ? 21 : 19); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
        if (MASKT) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmM) : "memory");
        if (KIND != WGRAD) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmO) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)),
                     "r"((uint32_t)TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // both CTAs' barriers exist before anything is signalled across the pair
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // K rows past the segment end in stage s's A and B tiles (two 64-column chunks each, the B tile directly behind the
    // A tile) := 0. Zeroing A alone would do for finite data (0 x finite = 0); B as well keeps a non-finite value of the
    // next segment out of this segment's sums.
    auto zero_tail = [&](int s, int valid) {
        const int nz = ((valid + 15) / 16) * 16 - valid;  // up to the end of the K step of 16 that holds the segment's end:
                                                           // the K steps behind it are not issued at all
        const int lines = nz * 4;
        for (int u = lane; u < lines * 8; u += 32) {
            const int line = u >> 3, part = u & 7;
            const int chunk = line / nz, krow = valid + line % nz;
            *reinterpret_cast<uint4 *>(smem + s * STAGE2_BYTES + chunk * (BK * 128) + krow * 128 + part * 16) =
                make_uint4(0, 0, 0, 0);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
    };
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0, mask_ph = 0;
            bool ok = true;
            PairTiles<KIND> it(p, dyn, (int32_t)cluster_id, (int32_t)n_clusters, sched_ring, sched_full0, sched_empty0, abort_flag, false, true);
            Tile t;
            // MASKT: the mask tile of a row tile can only land after the epilogue has read the previous one, which
            // happens while the next tile's K blocks are already being loaded: the load stays "due" and is issued
            // from the K loop as soon as the region is free, so the producer never stops to wait for the epilogue.
            bool mask_due = false;
            int mask_n0 = 0, mask_row0 = 0;
            auto load_mask = [&](bool blocking) -> bool {
                if (blocking) {
                    if (!mbar_wait(mempty_bar, mask_ph ^ 1u, abort_flag, p.status)) return false;
                } else if (!mbar_try_wait(mempty_bar, mask_ph ^ 1u)) {
                    return true;
                }
                const int nblk = min(4, (p.N - mask_n0) / 64);
                mbar_expect_tx(mfull_bar, nblk * 16384);
                for (int b = 0; b < nblk; ++b)
                    tma_load_2d(mask_smem + b * 16384, &tmM, mfull_bar, mask_n0 + b * 64, mask_row0 + 128 * (int)rank);
                mask_ph ^= 1u;
                mask_due = false;
                return true;
            };
            int trace_tile = -1;
            while (ok && it.next(t)) {
                int term = 0, kk = 0;  // ROW_*: piece of the contraction and column inside it
                ++trace_tile;
                long long tr_empty = 0;
                for (int kb = 0; kb < t.kblocks && ok; ++kb) {
                    if (MASKT && mask_due) load_mask(false);
                    const long long tw0 = TILE_CLOCK();
                    ok = mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status);
                    if (!ok) break;
                    tr_empty += TILE_CLOCK() - tw0;
                    if (kb == 0) TILE_TRACE_SET(0, trace_tile, 0, TILE_CLOCK());
                    if (kb == t.kblocks - 1) { TILE_TRACE_SET(0, trace_tile, 2, TILE_CLOCK()); TILE_TRACE_SET(0, trace_tile, 1, tr_empty); }
                    const uint32_t a_dst = base + s * STAGE2_BYTES, b_dst = a_dst + A2_BYTES;
                    if (KIND == WGRAD) {
                        const int r = t.row0 + kb * BK;
                        if (t.row_end - r < BK) {  // ragged last block: both tiles land on this CTA's own barrier first
                            if (rank == 0) mbar_expect_tx(full_bar(s), 0);  // nothing counts on the pair's barrier: the
                                                                            // "ready" barrier gates this stage
                            mbar_expect_tx(afull_bar(s), STAGE2_BYTES);
                            tma_load_3d(a_dst, &tmA, afull_bar(s), 0, r, t.m0 / 64 + 2 * (int)rank);
                            tma_load_3d(b_dst, &tmB, afull_bar(s), 0, r, t.b_chunk + 2 * (int)rank);
                        } else {
                            if (rank == 0) mbar_expect_tx(full_bar(s), 2 * STAGE2_BYTES);
                            tma2_load_3d(a_dst, &tmA, full_bar(s), 0, r, t.m0 / 64 + 2 * (int)rank);
                            tma2_load_3d(b_dst, &tmB, full_bar(s), 0, r, t.b_chunk + 2 * (int)rank);
                        }
                    } else {
                        if (rank == 0) mbar_expect_tx(full_bar(s), 2 * STAGE2_BYTES);
                        tma2_load_2d(a_dst, &tmA, full_bar(s), p.a_term_col[term] + kk, t.row0 + 128 * (int)rank);
                        if (KIND == ROW_BMN)
                            tma2_load_4d(b_dst, &tmB, full_bar(s), 0, p.b_term_col[term] + kk, t.n0 / 64 + 2 * (int)rank, t.e);
                        else
                            tma2_load_3d(b_dst, &tmB, full_bar(s), p.b_term_col[term] + kk, t.n0 + 128 * (int)rank, t.e);
                        kk += BK;
                        if (kk == p.K) { kk = 0; ++term; }
                    }
                    if (++s == NST) { s = 0; ph ^= 1u; }
                }
                if (MASKT && ok) {  // this tile's mask rows are due once the previous tile's have been read
                    if (mask_due) ok = load_mask(true);  // the previous tile's mask is still due: now it has to go
                    mask_due = ok;
                    mask_n0 = t.n0; mask_row0 = t.row0;
                    if (ok) load_mask(false);
                }
            }
            if (MASKT && ok && mask_due) load_mask(true);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even CTA only)
        // One thread runs the whole loop: nothing in it needs the other lanes, and a single-thread loop has no
        // divergence / reconvergence around the issue of every K block.
        if (rank == 0 && lane == 0) {
            constexpr uint32_t idesc = make_idesc2(KIND == WGRAD ? 1 : 0, KIND == ROW_BK ? 0 : 1);
            int s = 0, acc = 0;
            uint32_t ph = 0, acc_ph = 0, tail_ph = 0;  // tail_ph: one phase bit per stage for afull / ready
            bool ok = true;
            PairTiles<KIND> it(p, dyn, (int32_t)cluster_id, (int32_t)n_clusters, sched_ring, sched_full0, sched_empty0, abort_flag, false, true);
            Tile t;
            int trace_tile = -1;
            while (ok && it.next(t)) {
                ++trace_tile;
                if (t.kblocks == 0) continue;  // empty segment (WGRAD): the epilogue writes zeros
                TILE_TRACE_SET(1, trace_tile, 0, TILE_CLOCK());
                ok = mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
                TILE_TRACE_SET(1, trace_tile, 1, TILE_CLOCK());
                long long tr_wait = 0, tr_issue = 0;
                const uint32_t d_tmem = tmem_base + acc * BN;
                const int tail_valid = KIND == WGRAD ? (t.row_end - t.row0) - (t.kblocks - 1) * BK : BK;  // rows of the last block
                for (int kb = 0; kb < t.kblocks; ++kb) {
                    if (KIND == WGRAD && kb == t.kblocks - 1 && tail_valid < BK) {
                        const uint32_t tp = (tail_ph >> s) & 1u;  // fixed by warp 10 of both CTAs, ahead of time
                        ok = mbar_wait(ready_bar(s), tp, abort_flag, p.status) && mbar_try_wait_cluster(ready_bar(s), tp);
                        if (!ok) break;
                        tail_ph ^= 1u << s;
                    }
                    const long long tw0 = TILE_CLOCK();
                    ok = mbar_wait(full_bar(s), ph, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    tr_wait += TILE_CLOCK() - tw0;
                    const uint32_t a_src = base + s * STAGE2_BYTES, b_src = a_src + A2_BYTES;
                    const long long ti0 = TILE_CLOCK();
                    const uint64_t ad0 = KIND == WGRAD ? desc_mnmajor(a_src) : desc_kmajor(a_src);
                    const uint64_t bd0 = KIND == ROW_BK ? desc_kmajor(b_src) : desc_mnmajor(b_src);
                    // a K step of 16 advances the start address (low descriptor bits, in 16-byte units) by 32 bytes in a
                    // K-major tile and by 16 rows of 128 bytes in an MN-major one; the sum never leaves the address field
                    constexpr uint64_t a_step = KIND == WGRAD ? (16 * 128) >> 4 : 32 >> 4;
                    constexpr uint64_t b_step = KIND == ROW_BK ? 32 >> 4 : (16 * 128) >> 4;
                    const int ksteps = (KIND == WGRAD && kb == t.kblocks - 1) ? (tail_valid + 15) / 16 : BK / 16;
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        if (k < ksteps) tc_mma2_bf16(d_tmem, ad0 + k * a_step, bd0 + k * b_step, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                    tc_commit2(empty_bar(s));
                    tr_issue += TILE_CLOCK() - ti0;
                    if (++s == NST) { s = 0; ph ^= 1u; }
                }
                if (ok) tc_commit2(tfull_bar(acc));
                TILE_TRACE_SET(1, trace_tile, 3, TILE_CLOCK());
                TILE_TRACE_SET(1, trace_tile, 2, tr_wait); TILE_TRACE_SET(0, trace_tile, 3, tr_issue);
                if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
            }
        }
    } else if (warp == 11) {
        // ------------------------------------------------------------------ tile scheduler (even CTA, one thread)
        if (dyn && rank == 0 && lane == 0) {
            const uint32_t peer_ring = peer_smem_addr(sched_ring, 1), peer_full0 = peer_smem_addr(sched_full0, 1);
            bool ok = true;
            for (int i = 0; ok; ++i) {
                const int slot = i & (SCHED_SLOTS - 1);
                if (i >= SCHED_SLOTS) {  // every reader of the record this slot held has its copy
                    const uint32_t par = (uint32_t)(i / SCHED_SLOTS - 1) & 1u;
                    ok = mbar_wait(sched_empty0 + 8u * slot, par, abort_flag, p.status) && mbar_try_wait_cluster(sched_empty0 + 8u * slot, par);
                    if (!ok) break;
                }
                const int32_t id = atomicAdd(p.sched_counter, 1);
                int4 rec = make_int4(-1, 0, 0, 0);
                if (id < p.total_tiles) {
                    rec = p.sched_table[id / p.sched_group];
                    rec.w = id;
                }
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sched_ring + 16u * slot), "r"(rec.x), "r"(rec.y), "r"(rec.z), "r"(rec.w) : "memory");
                st_cluster_v4(peer_ring + 16u * slot, rec);
                mbar_arrive(sched_full0 + 8u * slot);
                mbar_arrive_cluster_addr(peer_full0 + 8u * slot);
                if (rec.x < 0) break;
            }
        }
    } else if (warp == 10) {
        // ------------------------------------------------------------------ WGRAD: ragged K tail (both CTAs)
        // The last K block of a segment holds rows of the next segment: they are zeroed in this CTA's A tile as soon as
        // it has landed, several stages before the MMAs get there, and reported on the even CTA's "ready" barrier.
        if (KIND == WGRAD) {
            int s = 0;
            uint32_t tail_ph = 0;
            bool ok = true;
            PairTiles<KIND> it(p, dyn, (int32_t)cluster_id, (int32_t)n_clusters, sched_ring, sched_full0, sched_empty0, abort_flag, true, lane == 0);
            Tile t;
            while (ok && it.next(t)) {
                for (int kb = 0; kb < t.kblocks; ++kb) {
                    const int valid = t.row_end - (t.row0 + kb * BK);
                    if (valid < BK) {
                        ok = mbar_wait(afull_bar(s), (tail_ph >> s) & 1u, abort_flag, p.status);
                        if (!ok) break;
                        zero_tail(s, valid);
                        if (lane == 0) mbar_arrive_leader(ready_bar(s));
                        __syncwarp();
                        tail_ph ^= 1u << s;
                    }
                    if (++s == NST) s = 0;
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
        const int quarter = warp & 3, half = (warp - 2) >> 2;
        const int pack_mode = p.bits_in ? 8 : (p.bias ? 1 : 0) | (p.relu ? 2 : 0) | (p.mask ? 4 : 0);
        uint8_t *stage_o = smem + NST * STAGE2_BYTES + (warp - 2) * 4096;
        uint32_t mask_ph = 0;
        int acc = 0;
        uint32_t acc_ph = 0;
        bool ok = true;
        PairTiles<KIND> it(p, dyn, (int32_t)cluster_id, (int32_t)n_clusters, sched_ring, sched_full0, sched_empty0, abort_flag, true, lane == 0);
        Tile t;
        int trace_tile = -1;
        while (ok && it.next(t)) {
            const bool have_acc = t.kblocks > 0;
            ++trace_tile;
            if (warp == 2 && lane == 0) TILE_TRACE_SET(2, trace_tile, 0, TILE_CLOCK());
            const uint4 bias_mine = bias_slice_load(p.bias, (int64_t)t.e * p.N, t.n0 + half * (BN / 2), p.N, lane);
            long long tr_ld = 0, tr_st = 0, tr_pack = 0;
            int64_t tile_row0, out_off = 0;
            int32_t rows_valid;
            if (KIND == WGRAD) {
                out_off = (int64_t)t.e * p.M * p.N;
                tile_row0 = t.m0 + 128 * (int)rank + quarter * 32;
                rows_valid = p.M - (int32_t)tile_row0;
            } else {
                tile_row0 = (int64_t)t.row0 + 128 * (int)rank + quarter * 32;
                rows_valid = t.row_end - (int32_t)tile_row0;
            }
            const int my_piece = lane & 7, my_sub = lane >> 3;
            const bool row_ok = lane < rows_valid;
            const int64_t out_row = tile_row0 + lane;
            uint4 keep4 = make_uint4(0, 0, 0, 0);  // the mask bits of this thread's row for the warp's four 32-column pieces
            if (p.bits_in && row_ok) {
                const uint32_t *kw = p.bits_in + out_row * (p.N >> 5) + ((t.n0 + half * (BN / 2)) >> 5);
                const int left = (p.N - (t.n0 + half * (BN / 2))) >> 5;  // words that exist in this row from here on
                if (left > 0) keep4.x = kw[0];
                if (left > 1) keep4.y = kw[1];
                if (left > 2) keep4.z = kw[2];
                if (left > 3) keep4.w = kw[3];
            }
            if (have_acc) {  // (the loads above are in flight while the warp waits for its accumulator)
                ok = mbar_wait(tfull_bar(acc), acc_ph, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
            }
            if (warp == 2 && lane == 0) TILE_TRACE_SET(2, trace_tile, 1, TILE_CLOCK());
            if (MASKT) {
                ok = mbar_wait(mfull_bar, mask_ph, abort_flag, p.status);
                if (!ok) break;
                mask_ph ^= 1u;
            }
            // Whole 32-row pieces go out as bulk tensor stores: each lane writes its row's 64-byte pieces into the
            // warp's own rows of a [128][64] block (the place the mask values were just read from, for MASKT), and one
            // lane stores each finished [32][64] box. Ragged pieces (segment end) use the guarded row stores.
            const bool staged = KIND != WGRAD && p.tma_out && !p.out_f32 && rows_valid >= 32;
            const int mrow = quarter * 32 + lane;
            if (staged && !MASKT) {  // the previous tile's boxes must have been read out of shared memory
                if (lane == 0) tma_store_wait_read();
                __syncwarp();
            }
            for (int c = half * (BN / 64); c < (half + 1) * (BN / 64); ++c) {
                const int col0 = t.n0 + c * 32;
                if (col0 >= p.N) break;
                uint32_t v[32];
                if (have_acc) {
                    const long long tl0 = TILE_CLOCK();
                    tc_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN + c * 32, v);
                    tc_ld_wait();
                    tr_ld += TILE_CLOCK() - tl0;
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                uint4 bias_raw[4];
                if (p.bias) bias_slice_piece(bias_mine, c - half * (BN / 64), bias_raw);  // whole warp: shuffles
                if (p.out_f32) {
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        *reinterpret_cast<uint4 *>(stage_o + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                            make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int row = 4 * i + my_sub;
                        if (row < rows_valid)
                            *reinterpret_cast<uint4 *>(p.out_f32 + out_off + (tile_row0 + row) * p.N + col0 + my_piece * 4) =
                                *reinterpret_cast<const uint4 *>(stage_o + row * 128 + ((my_piece ^ (row & 7)) << 4));
                    }
                    __syncwarp();
                } else if (row_ok || p.colsum_part) {  // with column sums the whole warp takes part (shuffles)
                    uint4 packed[4];
                    uint4 mask_raw[4];
                    if (MASKT) {  // from the tile in shared memory: row = this thread's row, 16-B pieces swizzled by row
                        const uint8_t *mrow_p = smem + NST * STAGE2_BYTES + (c >> 1) * 16384 + mrow * 128;
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            mask_raw[q] = *reinterpret_cast<const uint4 *>(mrow_p + ((((c & 1) * 4 + q) ^ (mrow & 7)) << 4));
                    } else if (p.mask && row_ok) {
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            mask_raw[q] = reinterpret_cast<const uint4 *>(p.mask + out_row * p.N + col0)[q];
                    }
                    const long long tp0 = TILE_CLOCK();
                    const int ci = c - half * (BN / 64);
                    pack32(pack_mode, v, bias_raw, mask_raw, packed, ci == 0 ? keep4.x : ci == 1 ? keep4.y : ci == 2 ? keep4.z : keep4.w);
                    if (p.bits_out && row_ok) p.bits_out[out_row * (p.N >> 5) + (col0 >> 5)] = positive_bits(packed);
                    tr_pack += TILE_CLOCK() - tp0;
                    if (staged) {
                        // with one box per warp (two [128][64] blocks, one per column half) the second box of a tile
                        // goes where the first one was: its bulk store must have read the box out first
                        uint8_t *blk = smem + NST * STAGE2_BYTES + (ONE_BOX ? half : (c >> 1)) * 16384;
                        if (ONE_BOX && (c & 3) == 2) {
                            if (lane == 0) tma_store_wait_read();
                            __syncwarp();
                        }
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            *reinterpret_cast<uint4 *>(blk + mrow * 128 + ((((c & 1) * 4 + q) ^ (mrow & 7)) << 4)) = packed[q];
                        if (c & 1) {  // the box of 64 columns is complete
                            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                            __syncwarp();
                            if (lane == 0) {
                                tma_store_2d(&tmO, smem_u32(blk + quarter * 4096), t.n0 + (c >> 1) * 64, (int)tile_row0);
                                tma_store_commit();
                            }
                        }
                    } else if (row_ok) {
                        const long long ts0 = TILE_CLOCK();
                        uint4 *dst = reinterpret_cast<uint4 *>(p.out + out_off + out_row * p.N + col0);
                        st_global_32B(dst, packed[0], packed[1]);  // two full 32-byte sectors per row piece
                        st_global_32B(dst + 2, packed[2], packed[3]);
                        tr_st += TILE_CLOCK() - ts0;
                    }
                    if (p.colsum_part) {  // sums of the rounded values, rows past the segment end count as 0
                        float a[32];
                        const uint32_t *pw = reinterpret_cast<const uint32_t *>(packed);
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            a[2 * j] = row_ok ? __uint_as_float(pw[j] << 16) : 0.0f;
                            a[2 * j + 1] = row_ok ? __uint_as_float(pw[j] & 0xffff0000u) : 0.0f;
                        }
                        const float sum = warp_column_sums(a, lane);
                        p.colsum_part[(int64_t)((t.mt * 2 + (int)rank) * 4 + quarter) * p.N + col0 + lane] = sum;
                    }
                }
            }
            if (have_acc) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_leader_relaxed(tempty_bar(acc));
                if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
            }
            if (warp == 2 && lane == 0) {
                TILE_TRACE_SET(2, trace_tile, 2, TILE_CLOCK());
                TILE_TRACE_SET(2, trace_tile, 3, tr_ld); TILE_TRACE_SET(2, trace_tile, 4, tr_st); TILE_TRACE_SET(2, trace_tile, 5, tr_pack);
            }
            if (MASKT) {  // the next mask tile may land once this warp's boxes have been read out
                __syncwarp();
                if (lane == 0) {
                    if (staged) tma_store_wait_read();
                    mbar_arrive(mempty_bar);
                }
            }
        }
        if (KIND != WGRAD && lane == 0) tma_store_wait_all();  // no bulk store may outlive the CTA's shared memory
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the pair's MMAs read both CTAs' shared memory: leave together
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS)
                     : "memory");
    }
}

// ------------------------------------------------------------------------------------------ host
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// bf16 tensor map; dims innermost first, strides (bytes) for dims 1.., box per dim; 128-B swizzle
int32_t make_map(CUtensorMap *tm, const void *base, int rank, const uint64_t *dims, const uint64_t *strides,
                 const uint32_t *box) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return MOE_ERR_CUDA;
    cuuint64_t gdim[5], gstr[4];
    cuuint32_t bx[5], es[5];
    for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides[i];
    CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), gdim, gstr, bx,
                    es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? MOE_OK : MOE_ERR_CUDA;
}

// rows x cols activations, K-major operand: box 64 (cols) x 128 (rows)
int32_t map_rows_kmajor(CUtensorMap *tm, const void *p, int64_t rows, int64_t cols) {
    const uint64_t dims[2] = {(uint64_t)cols, (uint64_t)rows}, str[1] = {(uint64_t)cols * 2};
    const uint32_t box[2] = {64, BM};
    return make_map(tm, p, 2, dims, str, box);
}
// rows x cols activations, MN-major operand (contraction over rows): dims (64, rows, cols/64)
int32_t map_rows_mnmajor(CUtensorMap *tm, const void *p, int64_t rows, int64_t cols, int chunks) {
    const uint64_t dims[3] = {64, (uint64_t)rows, (uint64_t)(cols / 64)}, str[2] = {(uint64_t)cols * 2, 128};
    const uint32_t box[3] = {64, BK, (uint32_t)chunks};
    return make_map(tm, p, 3, dims, str, box);
}
// per-expert weight [n, K, N] used as MN-major B: dims (64, K, N/64, n)
int32_t map_weight_mnmajor(CUtensorMap *tm, const void *p, int64_t n, int64_t K, int64_t N) {
    const uint64_t dims[4] = {64, (uint64_t)K, (uint64_t)(N / 64), (uint64_t)n};
    const uint64_t str[3] = {(uint64_t)N * 2, 128, (uint64_t)K * N * 2};
    const uint32_t box[4] = {64, BK, BN / 64, 1};
    return make_map(tm, p, 4, dims, str, box);
}
// per-expert weight [n, N, K] used as K-major B: dims (K, N, n)
int32_t map_weight_kmajor(CUtensorMap *tm, const void *p, int64_t n, int64_t N, int64_t K) {
    const uint64_t dims[3] = {(uint64_t)K, (uint64_t)N, (uint64_t)n};
    const uint64_t str[2] = {(uint64_t)K * 2, (uint64_t)N * K * 2};
    const uint32_t box[3] = {64, BN, 1};
    return make_map(tm, p, 3, dims, str, box);
}

GemmParams default_params() {
    GemmParams p;
    memset(&p, 0, sizeof(p));
    p.nterms = 1;
    p.segs_per_term = 1;
    return p;
}

// per-expert weight as B of the two-CTA kernel: each CTA of the pair loads 128 of the 256 columns
int32_t map_weight_mnmajor_half(CUtensorMap *tm, const void *p, int64_t n, int64_t K, int64_t N) {
    const uint64_t dims[4] = {64, (uint64_t)K, (uint64_t)(N / 64), (uint64_t)n};
    const uint64_t str[3] = {(uint64_t)N * 2, 128, (uint64_t)K * N * 2};
    const uint32_t box[4] = {64, BK, 2, 1};
    return make_map(tm, p, 4, dims, str, box);
}
int32_t map_weight_kmajor_half(CUtensorMap *tm, const void *p, int64_t n, int64_t N, int64_t K) {
    const uint64_t dims[3] = {(uint64_t)K, (uint64_t)N, (uint64_t)n};
    const uint64_t str[2] = {(uint64_t)K * 2, (uint64_t)N * K * 2};
    const uint32_t box[3] = {64, 128, 1};
    return make_map(tm, p, 3, dims, str, box);
}

int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

// Derived tile counts the device code divides by; ids are 32-bit.
template <int KIND, int TM> int32_t complete_params(GemmParams &q, int64_t max_tiles) {
    if (max_tiles >= ((int64_t)1 << 31) - ((int64_t)1 << 22)) return MOE_ERR_UNSUPPORTED;
    q.tiles_n = (int32_t)cdiv(q.N, BN);
    q.per_e = KIND == WGRAD ? (int32_t)cdiv(q.M, TM) * q.tiles_n : 1;
    q.total_tiles = (int32_t)max_tiles;
    q.kblocks_row = KIND == WGRAD ? 0 : q.nterms * (q.K / BK);
    return MOE_OK;
}

template <int KIND> int32_t launch(const CUtensorMap &tmA, const CUtensorMap &tmB, const GemmParams &p_in,
                                   int64_t max_tiles, cudaStream_t st) {
    GemmParams p = p_in;
    MOE_TRY((complete_params<KIND, BM>(p, max_tiles)));
    static bool configured = false;
    if (!configured) {
        MOE_CUDA(cudaFuncSetAttribute(grouped_gemm_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
        configured = true;
    }
    if (max_tiles <= 0) return MOE_OK;
    const unsigned grid = (unsigned)imin(max_tiles, sm_count());
    grouped_gemm_kernel<KIND><<<grid, NTHREADS, SMEM_BYTES, st>>>(tmA, tmB, p);
    MOE_LAUNCHED();
    return MOE_OK;
}

// The sub-block accumulating wgrad (float output): two operand stages + 128 KiB of running sums
constexpr int SMEM_ACC_BYTES = 2 * STAGE_BYTES + 1024 + 256 + 8 * 16384;
int32_t launch_acc_wgrad(const CUtensorMap &tmA, const CUtensorMap &tmB, const GemmParams &p_in, int64_t max_tiles,
                         cudaStream_t st) {
    GemmParams p = p_in;
    MOE_TRY((complete_params<WGRAD, BM>(p, max_tiles)));
    static bool configured = false;
    if (!configured) {
        MOE_CUDA(cudaFuncSetAttribute(grouped_gemm_kernel<WGRAD, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_ACC_BYTES));
        configured = true;
    }
    if (max_tiles <= 0) return MOE_OK;
    const unsigned grid = (unsigned)imin(max_tiles, sm_count());
    grouped_gemm_kernel<WGRAD, true><<<grid, NTHREADS, SMEM_ACC_BYTES, st>>>(tmA, tmB, p);
    MOE_LAUNCHED();
    return MOE_OK;
}

template <int KIND, bool MASKT = false>
int32_t launch2(const CUtensorMap &tmA, const CUtensorMap &tmB, const GemmParams &p_in, int64_t max_tiles,
                cudaStream_t st, const CUtensorMap *tmM = nullptr, const CUtensorMap *tmO = nullptr) {
    GemmParams p = p_in;
    p.tma_out = tmO != nullptr;
    MOE_TRY((complete_params<KIND, 256>(p, max_tiles)));
    static int max_clusters = 0;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.blockDim = dim3(NTHREADS2); cfg.dynamicSmemBytes = SMEM2_BYTES; cfg.stream = st;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    if (!max_clusters) {
        MOE_CUDA(cudaFuncSetAttribute(grouped_gemm2_kernel<KIND, MASKT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES));
        cfg.gridDim = dim3(2 * (sm_count() / 2));
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, grouped_gemm2_kernel<KIND, MASKT>, &cfg) != cudaSuccess || n <= 0) return MOE_ERR_CUDA;
        max_clusters = n;
    }
    if (max_tiles <= 0) return MOE_OK;
#ifdef MOE_TILE_TRACE
    {   // the launch whose index (counted over the two-CTA launches of the process) equals MOE_TRACE_LAUNCH records
        const char *env = getenv("MOE_TRACE_LAUNCH");
        p.trace = env && atoi(env) == g_trace_launch_no;
        ++g_trace_launch_no;
    }
#endif
    cfg.gridDim = dim3(2 * (unsigned)imin(max_tiles, max_clusters));
    MOE_CUDA(cudaLaunchKernelEx(&cfg, grouped_gemm2_kernel<KIND, MASKT>, tmA, tmB, tmM ? *tmM : tmA, tmO ? *tmO : tmA, p));
    MOE_LAUNCHED();
    return MOE_OK;
}

}  // namespace

bool tc_ffn_supported(const moe_config &c) {
    return c.act == MOE_BF16 && c.d % 64 == 0 && c.h % 64 == 0 && c.d >= 64 && c.h >= 64;
}

int64_t tc_tile_ws_ints(int64_t R, int64_t nseg);
int64_t tc_ffn_ws_bytes(const moe_config &c) { return (tc_tile_ws_ints((int64_t)c.T * c.k, c.n) * 4 + 255) & ~255ll; }

// The 256-row tiles of the two-CTA kernel pay off when the average segment fills them.
static bool use_two_cta(int64_t R, int32_t nseg, int32_t flags) {
    if (flags & MOE_FLAG_TC_ONE_CTA) return false;
    return R / (nseg > 0 ? nseg : 1) >= 384;
}

// C[rows, N] = epilogue(A[rows, K] . B_e) over the segments; B_e = W[e] as [K, N] (transposed = false)
// or as [N, K] read transposed (transposed = true).
// Tile table of a ragged row GEMM: tile_prefix[e] = number of tm-row tiles of the segments before e
// (tile_prefix[nseg] = total), and one record per M tile {segment, first row, segment end, 0}; records past
// the last tile carry segment -1. One block.
__global__ void __launch_bounds__(1024) tile_table_kernel(const int32_t *__restrict__ offsets, int32_t n, int32_t tm,
                                                          int32_t max_m, int32_t *__restrict__ tile_prefix,
                                                          int4 *__restrict__ info, int32_t *__restrict__ counter) {
    __shared__ int32_t warp_sum[32];
    __shared__ int32_t carry;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int32_t base = 0; base < n; base += 1024) {
        const int32_t e = base + threadIdx.x;
        const int32_t v = e < n ? (offsets[e + 1] - offsets[e] + tm - 1) / tm : 0;
        int32_t inc = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int32_t o = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += o;
        }
        if (lane == 31) warp_sum[w] = inc;
        __syncthreads();
        if (w == 0) {
            const int32_t sw = warp_sum[lane];
            int32_t si = sw;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int32_t o = __shfl_up_sync(0xffffffffu, si, off);
                if (lane >= off) si += o;
            }
            warp_sum[lane] = si - sw;
        }
        __syncthreads();
        const int32_t excl = carry + warp_sum[w] + inc - v;
        if (e < n) tile_prefix[e] = excl;
        __syncthreads();
        if (threadIdx.x == 1023) carry = excl + v;
        __syncthreads();
    }
    if (threadIdx.x == 0) tile_prefix[n] = carry;
    if (threadIdx.x == 0 && counter) *counter = 0;  // run-time tile counter of the GEMM that follows
    __syncthreads();  // the prefix (global memory, this block's own writes) is complete
    const int32_t total = carry;
    for (int32_t mt = threadIdx.x; mt < max_m; mt += 1024) {
        if (mt >= total) { info[mt] = make_int4(-1, 0, 0, 0); continue; }
        int lo = 0, hi = n;  // last e with tile_prefix[e] <= mt (empty segments share a prefix: take the last)
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (tile_prefix[mid] <= mt) lo = mid; else hi = mid;
        }
        info[mt] = make_int4(lo, offsets[lo] + (mt - tile_prefix[lo]) * tm, offsets[lo + 1], 0);
    }
}

// ints a tile table needs behind its [nseg + 1] prefix (records are 16 bytes, 16-byte aligned)
int64_t tc_tile_ws_ints(int64_t R, int64_t nseg) { return ((nseg + 1 + 3) & ~(int64_t)3) + 4 * (cdiv(R, 128) + nseg + 1); }
static int4 *tile_info_of(int32_t *tile_prefix, int32_t nseg) {
    return reinterpret_cast<int4 *>(tile_prefix + ((nseg + 1 + 3) & ~3));
}
// the int32 behind the last record of a table of tm = 256-row tiles (the table is sized for 128-row tiles)
static int32_t *tile_counter_of(int32_t *tile_prefix, int32_t nseg, int64_t R) {
    return reinterpret_cast<int32_t *>(tile_info_of(tile_prefix, nseg) + cdiv(R, 256) + nseg);
}
static int32_t launch_tile_table(const int32_t *offsets, int32_t nseg, int32_t tm, int64_t R, int32_t *tile_prefix,
                                 cudaStream_t st, int32_t *counter = nullptr) {
    tile_table_kernel<<<1, 1024, 0, st>>>(offsets, nseg, tm, (int32_t)(cdiv(R, tm) + nseg), tile_prefix,
                                          tile_info_of(tile_prefix, nseg), counter);
    MOE_LAUNCHED();
    return MOE_OK;
}

// Sum of the epilogue's 32-row column sums over each segment (bias gradient), G blocks per M tile.
// A thread block takes 64 columns of one segment: 16 column lanes (four adjacent columns each, 16-byte loads) by 16 row
// lanes; row lane q takes the blocks b = b0 + q, b0 + q + 16, ... (eight loads in flight: the largest expert of a skewed
// batch has over a thousand blocks and sets this kernel's duration) and the 16 sums are added in lane order: the
// result does not depend on timing.
__global__ void __launch_bounds__(256) colsum_blocks_final_kernel(const float *__restrict__ part, int32_t N,
                                                                  const int32_t *__restrict__ tile_prefix, int32_t G,
                                                                  bf16 *__restrict__ out) {
    __shared__ float4 sh[16][16];
    const int32_t e = blockIdx.x, q = threadIdx.x >> 4, cl = threadIdx.x & 15;
    const int32_t j = blockIdx.y * 64 + cl * 4;  // N is a multiple of 64
    const int32_t b0 = tile_prefix[e] * G, b1 = tile_prefix[e + 1] * G;
    float4 s = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    int32_t b = b0 + q;
    for (; b + 16 * 7 < b1; b += 16 * 8) {
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = *reinterpret_cast<const float4 *>(part + (int64_t)(b + 16 * u) * N + j);
#pragma unroll
        for (int u = 0; u < 8; ++u) { s.x += v[u].x; s.y += v[u].y; s.z += v[u].z; s.w += v[u].w; }
    }
    for (; b < b1; b += 16) {
        const float4 v = *reinterpret_cast<const float4 *>(part + (int64_t)b * N + j);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    sh[q][cl] = s;
    __syncthreads();
    if (q == 0) {
        float4 t = sh[0][cl];
#pragma unroll
        for (int u = 1; u < 16; ++u) { t.x += sh[u][cl].x; t.y += sh[u][cl].y; t.z += sh[u][cl].z; t.w += sh[u][cl].w; }
        __nv_bfloat162 o0 = __floats2bfloat162_rn(t.x, t.y), o1 = __floats2bfloat162_rn(t.z, t.w);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t *>(&o0); pk.y = *reinterpret_cast<uint32_t *>(&o1);
        *reinterpret_cast<uint2 *>(out + (int64_t)e * N + j) = pk;
    }
}

int64_t tc_colsum_part_floats(int64_t R, int32_t nseg, int32_t N) { return (cdiv(R, 128) * 4 + 8 * (int64_t)nseg + 8) * N; }

// colsum_part / colsum_out: if set, out's column sums per segment (a bias gradient) are formed in the epilogue
// and reduced into colsum_out [nseg, N]; colsum_part needs tc_colsum_part_floats(R, nseg, N) floats
int32_t tc_row_gemm(const void *A, const void *W, bool transposed, const int32_t *offsets, int32_t nseg, int64_t R,
                    int32_t N, int32_t K, void *out, const void *bias, const void *mask, int relu,
                    int32_t *tile_prefix, int32_t *status, cudaStream_t st, int32_t flags,
                    float *colsum_part = nullptr, void *colsum_out = nullptr, uint32_t *bits_out = nullptr,
                    const uint32_t *bits_in = nullptr) {
    if (R == 0) {
        if (colsum_out) MOE_CUDA(cudaMemsetAsync(colsum_out, 0, sizeof(bf16) * (size_t)nseg * N, st));
        return MOE_OK;
    }
    auto finish = [&](int32_t rc, int32_t G) -> int32_t {
        if (rc != MOE_OK || !colsum_out) return rc;
        colsum_blocks_final_kernel<<<dim3((unsigned)nseg, (unsigned)cdiv(N, 64)), 256, 0, st>>>(colsum_part, N, tile_prefix, G,
                                                                                                   (bf16 *)colsum_out);
        MOE_LAUNCHED();
        return MOE_OK;
    };
    CUtensorMap tmA, tmB;
    MOE_TRY(map_rows_kmajor(&tmA, A, R, K));
    GemmParams p = default_params();
    p.offsets = offsets; p.tile_prefix = tile_prefix; p.tile_info = tile_info_of(tile_prefix, nseg);
    p.nseg = nseg; p.M = 0; p.N = N; p.K = K; p.R = R;
    p.out = (bf16 *)out; p.bias = (const bf16 *)bias; p.mask = (const bf16 *)mask; p.relu = relu; p.status = status;
    p.bits_out = bits_out; p.bits_in = bits_in;
    if (bits_in) p.mask = nullptr;  // the bits replace the element-wise mask tensor
    p.colsum_part = colsum_out ? colsum_part : nullptr;
    if (use_two_cta(R, nseg, flags)) {  // segments long enough to fill 256-row tiles: SM pairs
        if (transposed) MOE_TRY(map_weight_kmajor_half(&tmB, W, nseg, N, K));
        else MOE_TRY(map_weight_mnmajor_half(&tmB, W, nseg, K, N));
        p.sched_counter = tile_counter_of(tile_prefix, nseg, R);  // tiles handed out at run time
        p.sched_table = p.tile_info;
        p.sched_group = (int32_t)cdiv(N, BN);
        MOE_TRY(launch_tile_table(offsets, nseg, 256, R, tile_prefix, st, p.sched_counter));
        const int64_t max_tiles2 = (cdiv(R, 256) + nseg) * cdiv(N, BN);
        CUtensorMap tmO;  // output rows as [32][64] boxes
        {
            const uint64_t dims[2] = {(uint64_t)N, (uint64_t)R};
            const uint64_t str[1] = {(uint64_t)N * 2};
            const uint32_t box[2] = {64, 32};
            MOE_TRY(make_map(&tmO, out, 2, dims, str, box));
        }
        if (transposed && mask && !bits_in) {  // the ReLU-mask rows come in as TMA tiles
            CUtensorMap tmM;
            MOE_TRY(map_rows_kmajor(&tmM, mask, R, N));
            return finish(launch2<ROW_BK, true>(tmA, tmB, p, max_tiles2, st, &tmM, &tmO), 8);
        }
        return finish(transposed ? launch2<ROW_BK>(tmA, tmB, p, max_tiles2, st, nullptr, &tmO)
                                 : launch2<ROW_BMN>(tmA, tmB, p, max_tiles2, st, nullptr, &tmO), 8);
    }
    if (transposed) MOE_TRY(map_weight_kmajor(&tmB, W, nseg, N, K));
    else MOE_TRY(map_weight_mnmajor(&tmB, W, nseg, K, N));
    MOE_TRY(launch_tile_table(offsets, nseg, BM, R, tile_prefix, st));
    const int64_t max_tiles = (cdiv(R, BM) + nseg) * cdiv(N, BN);
    return finish(transposed ? launch<ROW_BK>(tmA, tmB, p, max_tiles, st) : launch<ROW_BMN>(tmA, tmB, p, max_tiles, st), 4);
}

// Order in which the two-CTA weight-gradient GEMM hands out its tiles: seg[r] = {e, first row, end row, 0} for the
// segment of rank r by descending size (equal sizes by index), and the tile counter reset. One thread per segment.
constexpr int SCHED_MAX_SEG = 8192;
__global__ void __launch_bounds__(256) wgrad_schedule_kernel(const int32_t *__restrict__ offsets, int32_t n,
                                                             int4 *__restrict__ seg, int32_t *__restrict__ counter) {
    __shared__ int32_t cnt[SCHED_MAX_SEG];
    for (int32_t e = threadIdx.x; e < n; e += blockDim.x) cnt[e] = offsets[e + 1] - offsets[e];
    __syncthreads();
    const int32_t e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e == 0) *counter = 0;
    if (e >= n) return;
    const int32_t mine = cnt[e];
    int32_t rank = 0;
    for (int32_t o = 0; o < n; ++o) rank += (cnt[o] > mine || (cnt[o] == mine && o < e)) ? 1 : 0;
    seg[rank] = make_int4(e, offsets[e], offsets[e + 1], 0);
}

// dW[e] [M, N] = A_e^T . B_e, contraction over the rows of segment e; A [R, M], B [R, N].
// sched_ws: 4 + 4 * nseg ints (16-byte aligned) for the run-time tile order of the two-CTA kernel, or nullptr.
int32_t tc_wgrad_gemm(const void *A, const void *B, const int32_t *offsets, int32_t nseg, int64_t R, int32_t M,
                      int32_t N, void *out, int32_t *status, cudaStream_t st, int32_t flags, int32_t *sched_ws) {
    CUtensorMap tmA, tmB;
    GemmParams p = default_params();
    p.offsets = offsets; p.nseg = nseg; p.M = M; p.N = N; p.R = R;
    p.out = (bf16 *)out; p.status = status;
    if (use_two_cta(R, nseg, flags) && M >= 256) {  // SM pairs: 256 x 256 tiles, each CTA stages half of A and half of B
        MOE_TRY(map_rows_mnmajor(&tmA, A, R > 0 ? R : 1, M, 2));
        MOE_TRY(map_rows_mnmajor(&tmB, B, R > 0 ? R : 1, N, 2));
        if (sched_ws && nseg > 1 && nseg <= SCHED_MAX_SEG) {  // tiles of unequal length: longest first, handed out at run time
            p.sched_counter = sched_ws;
            p.sched_table = reinterpret_cast<const int4 *>(sched_ws + 4);
            p.sched_group = (int32_t)(cdiv(M, 256) * cdiv(N, BN));
            wgrad_schedule_kernel<<<(unsigned)cdiv(nseg, 256), 256, 0, st>>>(offsets, nseg, reinterpret_cast<int4 *>(sched_ws + 4),
                                                                          sched_ws);
            MOE_LAUNCHED();
        }
        return launch2<WGRAD>(tmA, tmB, p, (int64_t)nseg * cdiv(M, 256) * cdiv(N, BN), st);
    }
    MOE_TRY(map_rows_mnmajor(&tmA, A, R > 0 ? R : 1, M, BM / 64));
    MOE_TRY(map_rows_mnmajor(&tmB, B, R > 0 ? R : 1, N, BN / 64));
    return launch<WGRAD>(tmA, tmB, p, (int64_t)nseg * cdiv(M, BM) * cdiv(N, BN), st);
}

int32_t launch_tc_ffn(const moe_config &c, const void *xs, const int32_t *offsets, const void *W1, const void *b1,
                      const void *W2, const void *b2, void *hid, void *ys, void *ws, int32_t *status_word,
                      cudaStream_t st, bool first_only, uint32_t *relu_bits) {
    const int64_t R = (int64_t)c.T * c.k;
    int32_t *tile_prefix = static_cast<int32_t *>(ws);
    MOE_TRY(tc_row_gemm(xs, W1, false, offsets, c.n, R, c.h, c.d, hid, b1, nullptr, 1, tile_prefix, status_word, st, c.flags,
                        nullptr, nullptr, relu_bits));
    if (first_only) return MOE_OK;
    return tc_row_gemm(hid, W2, false, offsets, c.n, R, c.d, c.h, ys, b2, nullptr, 0, tile_prefix, status_word, st, c.flags);
}

// ------------------------------------------------------------------------------------------
// Gate backward contractions on the tensor cores (no bit-exactness is required there):
//   dW = x^T . dlogit   and   dX_gate = dlogit . [W_g | W_noise]^T
// with the float operands split into three bf16 terms (hi + mid + lo carries 24 mantissa bits), x being
// bf16 already. dsplit is [T, 3 * n2] = (hi | mid | lo) of the [T, n2] logit gradients (n2 = 2n: clean
// columns then raw-noise columns), wsplit is [d, 3 * n2] likewise for [W_g | W_noise].
// ------------------------------------------------------------------------------------------
// ldw: row stride of Wg and Wn in floats (n for two separate [d, n] matrices; 2n when they are the two halves of the
// columns of one [d, 2n] matrix)
__global__ void __launch_bounds__(256) split_weights_kernel(const float *__restrict__ Wg,
                                                            const float *__restrict__ Wn, int32_t d, int32_t n,
                                                            bf16 *__restrict__ wsplit, int32_t ldw) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int32_t n2 = 2 * n;
    if (i >= (int64_t)d * n2) return;
    const int32_t q = (int32_t)(i / n2), j = (int32_t)(i % n2);
    const float v = j < n ? Wg[(int64_t)q * ldw + j] : Wn[(int64_t)q * ldw + (j - n)];
    const bf16 hi = __float2bfloat16_rn(v);
    const float r1 = v - __bfloat162float(hi);
    const bf16 mid = __float2bfloat16_rn(r1);
    const bf16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
    bf16 *row = wsplit + (int64_t)q * 3 * n2;
    row[j] = hi; row[n2 + j] = mid; row[2 * n2 + j] = lo;
}

// out (group g = blockIdx.y) = sum_c part[c * part_stride + g * d * 2n + .], split into the W_g and W_noise halves
__global__ void __launch_bounds__(256) reduce_partials_kernel(const float *__restrict__ part, int32_t nparts,
                                                              int64_t part_stride, int32_t d, int32_t n,
                                                              float *__restrict__ dWg, float *__restrict__ dWn,
                                                              int32_t ldw) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int32_t n2 = 2 * n;
    const int64_t total = (int64_t)d * n2;
    if (i >= total) return;
    const int64_t g = blockIdx.y;
    double s = 0.0;
    for (int32_t c = 0; c < nparts; ++c) s += (double)part[(int64_t)c * part_stride + g * total + i];
    const int32_t q = (int32_t)(i / n2), j = (int32_t)(i % n2);
    if (j < n) dWg[(g * d + q) * ldw + j] = (float)s;
    else dWn[(g * d + q) * ldw + (j - n)] = (float)s;
}

bool tc_gate_bwd_supported(int32_t act, int32_t d, int32_t n) {
    // dX_gate contracts over the 2n logit columns (six split terms each) in one fp32 tensor-core accumulator, which
    // truncates: beyond 2n = 4096 the result drifts past 1e-5 (measured 2e-5 at n = 8192), so very wide flat gates take
    // the fp32 SIMT contractions instead
    return act == MOE_BF16 && d % 64 == 0 && (2 * n) % 64 == 0 && 2 * n <= 4096;
}

// dW of the gate: the contraction over the tokens is cut into row ranges (one float partial per range and precision
// term, added in double afterwards), and inside a range the tensor-core accumulator is restarted every GB_ROWS_HI rows
// for the leading (hi) term: an fp32 accumulator loses low bits when a long run of same-sign terms is added (e.g. the
// gradient of a constant input feature); 128 rows keep that below 1e-5 of the result. The mid and lo terms are 2^-8
// and 2^-16 of the hi term and restart every GB_ROWS_LO rows. The restarts' sums are added in shared memory (see the
// ACC kernel), so only one partial per range goes to global memory.
constexpr int GB_ROWS_HI = 128, GB_ROWS_LO = 2048;
static void gate_bwd_split(int64_t T, int32_t d, int32_t n, int32_t *nranges, int32_t *rows) {
    const int64_t tiles_per_range = cdiv(d, BM) * cdiv(2 * n, BN);
    int64_t want = cdiv(3 * (int64_t)sm_count(), tiles_per_range);  // about three waves of hi-term tiles
    const int64_t most = T > 0 ? cdiv(T, GB_ROWS_LO) : 1;
    if (want > most) want = most;
    if (want < 1) want = 1;
    const int64_t r = cdiv(cdiv(T > 0 ? T : 1, want), GB_ROWS_LO) * GB_ROWS_LO;  // whole lo sub-blocks per range
    *rows = (int32_t)r;
    *nranges = (int32_t)(T > 0 ? cdiv(T, r) : 1);
}

int64_t tc_gate_bwd_partials(int64_t T, int32_t d, int32_t n) {
    int32_t nr, rows;
    gate_bwd_split(T, d, n, &nr, &rows);
    return (int64_t)3 * nr * d * 2 * n;
}

int32_t launch_tc_gate_bwd(const void *x, int64_t T, int32_t d, int32_t n, const float *Wg, const float *Wn,
                           const void *dsplit, void *wsplit, float *partials, float *dWg, float *dWn,
                           float *dX_gate, int32_t *status, cudaStream_t st, int32_t flags, int32_t ldw) {
    const int32_t n2 = 2 * n;
    if (T == 0 && ldw > 0) {
        for (int32_t q = 0; q < d; ++q) MOE_CUDA(cudaMemsetAsync(dWg + (int64_t)q * ldw, 0, sizeof(float) * n2, st));
        return MOE_OK;
    }
    if (T == 0) {
        MOE_CUDA(cudaMemsetAsync(dWg, 0, sizeof(float) * d * n, st));
        MOE_CUDA(cudaMemsetAsync(dWn, 0, sizeof(float) * d * n, st));
        return MOE_OK;
    }
    split_weights_kernel<<<(unsigned)cdiv((int64_t)d * n2, 256), 256, 0, st>>>(Wg, Wn, d, n, (bf16 *)wsplit, ldw > 0 ? ldw : n);
    MOE_LAUNCHED();
    int32_t nr, rows;
    gate_bwd_split(T, d, n, &nr, &rows);
    {   // dW partials: contraction over the tokens, cut into row ranges, one set per precision term
        CUtensorMap tmA, tmB;
        MOE_TRY(map_rows_mnmajor(&tmA, x, T, d, BM / 64));
        MOE_TRY(map_rows_mnmajor(&tmB, dsplit, T, 3 * n2, BN / 64));
        GemmParams p = default_params();
        p.nseg = 3 * nr; p.M = d; p.N = n2; p.R = T; p.out_f32 = partials; p.status = status;
        p.segs_term0 = nr; p.rows_per_seg0 = rows;
        p.rows_per_seg = rows; p.segs_per_term = nr; p.b_term_chunks = n2 / 64;
        p.sub_kb0 = GB_ROWS_HI / BK; p.sub_kb = GB_ROWS_LO / BK; p.interleave = 3;
        MOE_TRY(launch_acc_wgrad(tmA, tmB, p, (int64_t)p.nseg * cdiv(d, BM) * cdiv(n2, BN), st));
        reduce_partials_kernel<<<(unsigned)cdiv((int64_t)d * n2, 256), 256, 0, st>>>(partials, 3 * nr, (int64_t)d * n2, d, n, dWg, dWn,
                                                                                     ldw > 0 ? ldw : n);
        MOE_LAUNCHED();
    }
    {   // dX_gate: six cross terms of the two split operands, concatenated along the contraction
        CUtensorMap tmA, tmB;
        const bool pairs = T >= 256 * 74 && !(flags & MOE_FLAG_TC_ONE_CTA);  // enough 256-row tiles for every SM pair
        MOE_TRY(map_rows_kmajor(&tmA, dsplit, T, 3 * n2));
        if (pairs) MOE_TRY(map_weight_kmajor_half(&tmB, wsplit, 1, d, 3 * n2));
        else MOE_TRY(map_weight_kmajor(&tmB, wsplit, 1, d, 3 * n2));
        GemmParams p = default_params();
        p.nseg = 1; p.N = d; p.K = n2; p.R = T; p.out_f32 = dX_gate; p.status = status;
        p.nterms = 6;
        const int32_t at[6] = {2, 0, 1, 0, 1, 0}, bt[6] = {0, 2, 1, 1, 0, 0};  // smallest products first
        for (int i = 0; i < 6; ++i) { p.a_term_col[i] = at[i] * n2; p.b_term_col[i] = bt[i] * n2; }
        if (pairs) MOE_TRY(launch2<ROW_BK>(tmA, tmB, p, cdiv(T, 256) * cdiv(d, BN), st));
        else MOE_TRY(launch<ROW_BK>(tmA, tmB, p, cdiv(T, BM) * cdiv(d, BN), st));
    }
    return MOE_OK;
}

// Forward gate projection for the routing screen: cr = x . (W_lo + W_mid + W_hi), smallest term first.
bool tc_gate_fwd_supported(int32_t act, int64_t T, int32_t d, int32_t n, int32_t flags) {
    // MOE_FLAG_GATE_SCREEN_OFF: every token through the fma chain; _ON: screen whenever the shapes allow;
    // neither: screen when the projection is large enough to pay for the extra launches
    if (flags & MOE_FLAG_GATE_SCREEN_OFF) return false;
    if (!(act == MOE_BF16 && d % 64 == 0 && (2 * n) % 64 == 0 && T >= 256)) return false;
    if (flags & MOE_FLAG_GATE_SCREEN_ON) return true;
    return (double)T * d * 2.0 * n >= 1.0e9;
}

int32_t launch_tc_gate_fwd(const void *x, int64_t T, int32_t d, int32_t n, const void *wsplit, float *cr,
                           int32_t *status, cudaStream_t st) {
    const int32_t n2 = 2 * n;
    CUtensorMap tmA, tmB;
    MOE_TRY(map_rows_kmajor(&tmA, x, T, d));
    MOE_TRY(map_weight_mnmajor_half(&tmB, wsplit, 1, 3 * (int64_t)d, n2));
    GemmParams p = default_params();
    p.nseg = 1; p.N = n2; p.K = d; p.R = T; p.out_f32 = cr; p.status = status;
    p.nterms = 3;
    for (int i = 0; i < 3; ++i) { p.a_term_col[i] = 0; p.b_term_col[i] = (2 - i) * d; }
    return launch2<ROW_BMN>(tmA, tmB, p, cdiv(T, 256) * cdiv(n2, BN), st);
}

// The same for the secondary gates of the hierarchical layer: rows = the slots (t, s1) sorted by primary group
// (xs_p [P1, d], offsets_p [a + 1]), one [d, 2b] weight pair per group. wsplit_s [3][a * d][2b] (term, group, feature);
// cr_s [P1, 2b] comes out in sorted order.
int32_t launch_tc_gate_fwd_grouped(const void *xs_p, int64_t P1, int32_t d, int32_t a, int32_t b, const void *wsplit_s,
                                   const int32_t *offsets_p, int32_t *tile_prefix, float *cr_s, int32_t *status,
                                   cudaStream_t st, int32_t flags) {
    if (P1 == 0) return MOE_OK;
    const int32_t n2 = 2 * b;
    const bool pairs = use_two_cta(P1, a, flags);
    CUtensorMap tmA, tmB;
    MOE_TRY(map_rows_kmajor(&tmA, xs_p, P1, d));
    {   // the group is the map's last coordinate (stride d rows), the precision term an offset of a * d rows along K
        const uint64_t dims[4] = {64, (uint64_t)3 * a * d, (uint64_t)(n2 / 64), (uint64_t)a};
        const uint64_t str[3] = {(uint64_t)n2 * 2, 128, (uint64_t)d * n2 * 2};
        const uint32_t box[4] = {64, BK, pairs ? 2u : (uint32_t)(BN / 64), 1};
        MOE_TRY(make_map(&tmB, wsplit_s, 4, dims, str, box));
    }
    GemmParams p = default_params();
    p.offsets = offsets_p; p.tile_prefix = tile_prefix; p.tile_info = tile_info_of(tile_prefix, a);
    p.nseg = a; p.N = n2; p.K = d; p.R = P1; p.out_f32 = cr_s; p.status = status;
    p.nterms = 3;
    for (int i = 0; i < 3; ++i) { p.a_term_col[i] = 0; p.b_term_col[i] = (2 - i) * a * d; }  // lo, mid, hi
    const int32_t tm = pairs ? 256 : BM;
    MOE_TRY(launch_tile_table(offsets_p, a, tm, P1, tile_prefix, st));
    const int64_t max_tiles = (cdiv(P1, tm) + a) * cdiv(n2, BN);
    return pairs ? launch2<ROW_BMN>(tmA, tmB, p, max_tiles, st) : launch<ROW_BMN>(tmA, tmB, p, max_tiles, st);
}

// Secondary gates of the hierarchical layer: the slots (t, s1) sorted by primary group are the rows.
// xs_p [P1, d] token rows in sorted order, dsplit_s [P1, 3 * 2b] split logit gradients in sorted order.
bool tc_hier_gate_bwd_supported(int32_t act, int32_t d, int32_t a, int32_t b) {
    return act == MOE_BF16 && d % 64 == 0 && (2 * a) % 64 == 0 && (2 * b) % 64 == 0;
}

int32_t launch_tc_hier_secondary_bwd(const void *xs_p, const void *dsplit_s, void *wsplit_s, const float *Wg_s,
                                     const float *Wn_s, const int32_t *offsets_p, int32_t *tile_prefix, int32_t a,
                                     int64_t P1, int32_t d, int32_t b, float *partials, float *dWg_s, float *dWn_s,
                                     float *dX_sec, int32_t *status, cudaStream_t st) {
    const int32_t n2 = 2 * b;
    split_weights_kernel<<<(unsigned)cdiv((int64_t)a * d * n2, 256), 256, 0, st>>>(Wg_s, Wn_s, a * d, b, (bf16 *)wsplit_s, b);
    MOE_LAUNCHED();
    {   // dW_s[i] = sum over the slots of group i of x[token]^T . dlogit[slot], one partial per precision term
        CUtensorMap tmA, tmB;
        MOE_TRY(map_rows_mnmajor(&tmA, xs_p, P1 > 0 ? P1 : 1, d, BM / 64));
        MOE_TRY(map_rows_mnmajor(&tmB, dsplit_s, P1 > 0 ? P1 : 1, 3 * n2, BN / 64));
        GemmParams p = default_params();
        p.offsets = offsets_p; p.nseg = 3 * a; p.off_mod = a; p.b_term_chunks = n2 / 64;
        p.M = d; p.N = n2; p.R = P1; p.out_f32 = partials; p.status = status;
        MOE_TRY(launch<WGRAD>(tmA, tmB, p, (int64_t)p.nseg * cdiv(d, BM) * cdiv(n2, BN), st));
        reduce_partials_kernel<<<dim3((unsigned)cdiv((int64_t)d * n2, 256), (unsigned)a), 256, 0, st>>>(
            partials, 3, (int64_t)a * d * n2, d, b, dWg_s, dWn_s, b);
        MOE_LAUNCHED();
    }
    if (P1 > 0) {   // dX_sec[row] = dlogit[row] . [W_g | W_noise][group]^T, six cross terms
        CUtensorMap tmA, tmB;
        MOE_TRY(map_rows_kmajor(&tmA, dsplit_s, P1, 3 * n2));
        MOE_TRY(map_weight_kmajor(&tmB, wsplit_s, a, d, 3 * n2));
        MOE_TRY(launch_tile_table(offsets_p, a, BM, P1, tile_prefix, st));
        GemmParams p = default_params();
        p.offsets = offsets_p; p.tile_prefix = tile_prefix; p.tile_info = tile_info_of(tile_prefix, a);
        p.nseg = a; p.N = d; p.K = n2; p.R = P1;
        p.out_f32 = dX_sec; p.status = status;
        p.nterms = 6;
        const int32_t at[6] = {2, 0, 1, 0, 1, 0}, bt[6] = {0, 2, 1, 1, 0, 0};
        for (int i = 0; i < 6; ++i) { p.a_term_col[i] = at[i] * n2; p.b_term_col[i] = bt[i] * n2; }
        MOE_TRY(launch<ROW_BK>(tmA, tmB, p, (cdiv(P1, BM) + a) * cdiv(d, BN), st));
    }
    return MOE_OK;
}

int32_t launch_tc_ffn_bwd(const moe_config &c, const void *xs, const void *hid, const void *dys,
                          const int32_t *offsets, const void *W1, const void *W2, void *dxs, void *dW1, void *db1,
                          void *dW2, void *db2, void *dz, float *colsum, int32_t *tile_prefix, int32_t *status_word,
                          cudaStream_t st, const uint32_t *relu_bits) {
    const int64_t R = (int64_t)c.T * c.k;
    MOE_TRY(launch_segment_colsum(dys, c.act, offsets, c.n, R, c.d, db2, colsum, tile_prefix, st));
    MOE_TRY(tc_wgrad_gemm(hid, dys, offsets, c.n, R, c.h, c.d, dW2, status_word, st, c.flags, tile_prefix));
    // db1 = column sums of dz, formed in the epilogue of the GEMM that produces dz
    MOE_TRY(tc_row_gemm(dys, W2, true, offsets, c.n, R, c.h, c.d, dz, nullptr, hid, 0, tile_prefix, status_word, st, c.flags, colsum, db1,
                        nullptr, relu_bits));
    MOE_TRY(tc_wgrad_gemm(xs, dz, offsets, c.n, R, c.d, c.h, dW1, status_word, st, c.flags, tile_prefix));
    return tc_row_gemm(dz, W1, true, offsets, c.n, R, c.d, c.h, dxs, nullptr, nullptr, 0, tile_prefix, status_word, st, c.flags);
}

// ------------------------------------------------------------------------------------------
// The expiry path of the bounded waits, exercised on its own: one thread waits, with the helper the GEMM kernels use,
// on an mbarrier nobody arrives at. Nothing asynchronous is outstanding (no copy, no MMA, no tensor memory), so the
// kernel simply returns once the limit has passed and leaves MOE_ERR_TIMEOUT in the status word.
// ------------------------------------------------------------------------------------------
__global__ void debug_wait_kernel(int32_t *status, unsigned long long limit_ns) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_wait_limit(smem_u32(&bar), 0, &abort_flag, status, limit_ns);
}

int32_t launch_debug_wait(int32_t *status, unsigned long long limit_ns, cudaStream_t st) {
    debug_wait_kernel<<<1, 1, 0, st>>>(status, limit_ns);
    MOE_LAUNCHED();
    return MOE_OK;
}

MOE_BOUNDS_READER(bounds_violations_ffn)

}  // namespace moe

#ifdef MOE_TILE_TRACE
extern "C" int32_t moe_debug_tile_trace(long long *host_out) {
    return cudaMemcpyFromSymbol(host_out, moe::g_tile_trace, sizeof(moe::g_tile_trace)) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
#endif
