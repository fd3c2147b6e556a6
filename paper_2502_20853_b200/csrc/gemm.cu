// Block-scaled MXFP4 GEMM for sm_100a:  D[M,N] = deq(A)[M,Kc] * deq(B)[N,Kc]^T  (Eq. 3-5).
//
// One persistent, warp-specialised CTA per SM (12 warps):
//   warp 0      TMA producer: packed E2M1 tiles (128B-swizzled, 256 K elements per stage) -> shared-memory ring
//   warp 1      MMA issuer: tcgen05.mma kind::mxf4.block_scale, FP32 accumulators in TMEM; owns the TMEM
//               allocation
//   warp 2      scale copier: tcgen05.cp (scales smem -> TMEM).  tcgen05 operations of ONE thread run in
//               order, so copies issued by the MMA thread would stall its MMAs; from a thread of their own
//               they overlap them completely.  Each ring stage has its own scale columns in TMEM.
//   warp 3      second producer: the scale chunks (issuing an asynchronous copy costs its thread ~100 ns, a stage needs five)
//   warps 4-11  epilogue: tcgen05.ld -> (+bias) -> cast -> swizzled staging in shared memory -> TMA store;
//               two warps share each quarter of the TMEM lanes and split the columns
// Every mbarrier wait is bounded; on expiry MXFP4_DEV_TIMEOUT is raised and all roles drain.
#include "common.cuh"
#include "quant_tile.cuh"
#include "tma.cuh"

namespace mx {

constexpr int kBM = 128;           // rows of A per tile (one UMMA M)
constexpr int kBKBytes = 128;      // packed bytes of K per stage = 256 elements = one 128B swizzle atom
constexpr int kBKElems = 256;
constexpr int kMmaKBytes = 32;     // one tcgen05.mma kind::mxf4 consumes K = 64 elements = 32 bytes
constexpr int kSfChunk = 512;      // scales of 128 rows x 4 blocks (= 128 K elements)
constexpr int kEpiWarp0 = 4;       // first epilogue warp
constexpr int kEpiWarps = 8;
constexpr int kGemmThreads = 32 * (kEpiWarp0 + kEpiWarps);
constexpr int kStagingBytes = 2048;             // per epilogue warp: 32 rows x 64 bytes

// DEEP = false: the longest ring, one staging buffer per epilogue warp (long K loops).
// DEEP = true : a shorter ring and four staging buffers per epilogue warp, so that a warp can drain its part of the
//               accumulator without waiting for its own stores (short K loops, where the epilogue is the larger part).
template <int BN, bool DEEP>
struct GemmCfg {
    static constexpr int kRB = (BN + 127) / 128;                        // 128-row scale blocks of B per tile
    static constexpr int kABytes = kBM * kBKBytes;                      // 16 KB
    static constexpr int kBBytes = BN * kBKBytes;
    static constexpr int kSfaBytes = 2 * kSfChunk;                      // two K chunks of 128 elements
    static constexpr int kSfbBytes = 2 * kSfChunk * kRB;
    static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;
    static constexpr int kStages = BN <= 128 ? (DEEP ? 4 : 6) : BN <= 192 ? 4 : (DEEP ? 3 : 4);
    static constexpr int kStagingBufs = BN == 192 ? 3 : (DEEP ? (BN / 64) : 1);   // DEEP / 192: one buffer per 32-column chunk of a warp's share
    static constexpr int kAccStages = (BN <= 192) ? 2 : 1;              // tiles up to 192 wide leave room for two accumulators
    static constexpr int kSfCol = kAccStages * BN;                      // TMEM columns: accumulators, then per ring stage SFA (8) + SFB (8 kRB)
    static constexpr int kSfSlot = 8 + 8 * kRB;
    static constexpr int kTmemCols = 512;
    static constexpr int kStagingOff = kStages * kStageBytes;           // multiple of 1024
    static constexpr int kBarOff = kStagingOff + kEpiWarps * kStagingBufs * kStagingBytes;
    static constexpr int kSmemBytes = kBarOff + 1024 /*align*/ + 256 /*barriers*/;
    static_assert(kSfCol + kStages * kSfSlot <= 512, "TMEM budget");
    static_assert(kStageBytes % 1024 == 0, "stage alignment");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

struct GemmParams {
    const uint8_t *sfa;   // scales of A, tiled order
    const uint8_t *sfb;
    int64_t M, N, Kc;
    int nblk4;            // ceil(Kc/32/4): 512-byte chunks per 128-row block
    int rbA, rbB;         // 128-row scale blocks present in A / B buffers
    int tiles_m, tiles_n, splits, kt_total, kt_per_split;
    int out_fp32;         // element type of the stored tile (FP32 also for split-K partials)
    const __nv_bfloat16 *bias;   // applied only when splits == 1 (and by the cluster kernel, whose sum is complete)
    uint32_t *dev_status;
    void *d;              // the caller's output and its leading dimension (cluster kernel: plain stores)
    int64_t ldd;
    uint32_t spin_limit;  // polls after which a bounded wait gives up (kWaitSpinLimit in normal use)
    int withhold_loads;   // self-test of the drain path: the producers issue nothing, so every wait runs out
};

// ---- PTX wrappers of the tensor-core instructions (mbarrier, TMA and elect wrappers: tma.cuh) ----
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_cp_sf(uint32_t taddr, uint64_t sdesc)
{
    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void tc_mma_mxf4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t sfa_tmem,
                                            uint32_t sfb_tmem, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (sm_100 format, version 1).
//   K-major operand tile, rows of 128 bytes, 128B swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t desc_operand_sw128(uint32_t saddr)
{
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
//   Scale chunk: 32 rows x 16 bytes, no swizzle: 8-row core matrices are 128 bytes apart.
__device__ __forceinline__ uint64_t desc_sf(uint32_t saddr)
{
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(128u >> 4) << 32) | (1ull << 46);
}
// Instruction descriptor of kind::mxf4 (block scaled): E2M1 x E2M1, UE8M0 scales, K-major A and B, M = 128.
__device__ __forceinline__ uint32_t idesc_mxf4(int n, uint32_t a_sf_id, uint32_t b_sf_id)
{
    return (b_sf_id << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | (1u << 23) | ((uint32_t)(kBM >> 4) << 24) |
           (a_sf_id << 29);
}

// bias[0 .. ncols) (bf16, ncols a multiple of 8, at most N) added to v[0 .. N)
template <int N>
__device__ __forceinline__ void add_bias(float (&v)[N], const __nv_bfloat16 *bias, int ncols)
{
#pragma unroll
    for (int j = 0; j < N; j += 8) {
        if (j >= ncols) break;
        const uint4 b = __ldg(reinterpret_cast<const uint4 *>(bias + j));
        const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int t = 0; t < 4; t++) {
            v[j + 2 * t] += bf16lo(bw[t]);
            v[j + 2 * t + 1] += bf16hi(bw[t]);
        }
    }
}

// 32 accumulator columns of one row -> 32 bf16 in 16 words
__device__ __forceinline__ void pack_row_bf16(const uint32_t (&r)[32], const __nv_bfloat16 *bias, int ncols, uint32_t (&w)[16])
{
    float v[32];
#pragma unroll
    for (int j = 0; j < 32; j++) v[j] = __uint_as_float(r[j]);
    if (bias) add_bias<32>(v, bias, ncols);
#pragma unroll
    for (int j = 0; j < 16; j++) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
        w[j] = *reinterpret_cast<uint32_t *>(&h);
    }
}

// One row's 64 bytes into its staging line, in the 64B swizzle the TMA store expects: 16-byte chunk j of row r sits at
// chunk j ^ ((r >> 1) & 3).
__device__ __forceinline__ void stage_line(uint8_t *line, int row, const uint32_t *w /*16 words*/)
{
    const int sw = (row >> 1) & 3;
#pragma unroll
    for (int j = 0; j < 4; j++)
        *reinterpret_cast<uint4 *>(line + ((j ^ sw) << 4)) = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
}

// One row's 128 bytes (two 32-column chunks of bf16) into its line of a 128B-swizzled box: 16-byte piece j of row r sits
// at piece j ^ (r & 7).
__device__ __forceinline__ void stage_line_wide(uint8_t *line, int row, const uint32_t *w0 /*16 words*/, const uint32_t *w1)
{
    const int sw = row & 7;
#pragma unroll
    for (int j = 0; j < 4; j++) {
        *reinterpret_cast<uint4 *>(line + ((j ^ sw) << 4)) = make_uint4(w0[4 * j], w0[4 * j + 1], w0[4 * j + 2], w0[4 * j + 3]);
        *reinterpret_cast<uint4 *>(line + (((j + 4) ^ sw) << 4)) = make_uint4(w1[4 * j], w1[4 * j + 1], w1[4 * j + 2], w1[4 * j + 3]);
    }
}

// ---- epilogue of one tile for one warp -----------------------------------------------------------------
// The warp owns TMEM lanes (= tile rows) row0 .. row0 + 31 and BN / 2 accumulator columns starting at `taddr`
// (global column `colbase`).  bf16: the whole share is read and packed first, the accumulator is handed back (an
// arrive on `acc_empty_bar`), then the rows go through 64B-swizzled staging buffers to TMA stores clipped at M, N.
// `map_w` (bf16 only, may be null): the same output with boxes of 64 columns and 128B swizzle; pairs of chunks then
// leave through one store instead of two (issuing a store costs its thread about 150 cycles).
// Arrive on a barrier of another CTA of the cluster (a shared::cluster address).  Used to hand an accumulator back: what
// the arrive has to order are this warp's accumulator reads, which tcgen05.wait::ld has already completed, so the default
// semantics (release at CTA scope) do; a release at cluster scope costs the arriving thread 2500-4000 cycles while the
// memory system is busy (measured), which made the epilogue the slowest role of the two-CTA kernels.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

// REMOTE: `acc_empty_bar` is a shared::cluster address (the barrier lives in the leader of a CTA pair).
template <int BN, int BUFS, bool REMOTE = false>
__device__ __forceinline__ void epilogue_tile(const CUtensorMap *map_d, const CUtensorMap *map_w, const GemmParams &p, uint32_t taddr,
                                              int row0, int colbase, int split, uint8_t *staging, uint32_t &sbuf, int lane,
                                              uint32_t acc_empty_bar)
{
    constexpr int kHalfCols = BN / 2;
    constexpr int kChunks = kHalfCols / 32;
    const bool use_bias = p.bias != nullptr && p.splits == 1;
    // one staged 64-byte-wide box (32 rows) -> global
    auto store_box = [&](const uint32_t *w, int x) {
        // the store that last used this staging buffer must have finished reading it
        if (lane == 0) bulk_wait_read<BUFS - 1>();
        __syncwarp();
        uint8_t *buf = staging + sbuf * kStagingBytes;
        stage_line(buf + lane * 64, lane, w);
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
            tma_store_3d(map_d, x, row0, split, smem_u32(buf));
            bulk_commit();
        }
        sbuf = (sbuf + 1) % BUFS;
    };
    auto release_acc = [&]() {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
            if (REMOTE) mbar_arrive_remote(acc_empty_bar);
            else mbar_arrive(acc_empty_bar);
        }
    };
    if (!p.out_fp32) {
        // bf16: read and pack the warp's whole share first, hand the accumulator back, then store
        uint32_t pk[kChunks][16];
#pragma unroll
        for (int cc = 0; cc < kChunks; cc++) {
            const int col = colbase + cc * 32;
            if (col < p.N && row0 < p.M) {     // uniform across the warp; nothing to store otherwise
                uint32_t r[32];
                tc_ld32(taddr + cc * 32, r);
                tc_wait_ld();
                pack_row_bf16(r, use_bias ? p.bias + col : nullptr, (int)min((int64_t)32, p.N - col), pk[cc]);
            }
        }
        release_acc();
        if (BUFS >= kChunks && map_w != nullptr) {
            // as below, with each pair of chunks staged as one 128-byte-wide box (two staging buffers are contiguous)
            if (lane == 0) bulk_wait_read<0>();
            __syncwarp();
#pragma unroll
            for (int cc = 0; cc < kChunks; cc += 2) {
                if (colbase + cc * 32 < p.N && row0 < p.M) {
                    if (cc + 1 < kChunks) stage_line_wide(staging + cc * kStagingBytes + lane * 128, lane, pk[cc], pk[cc + 1 < kChunks ? cc + 1 : cc]);
                    else stage_line(staging + cc * kStagingBytes + lane * 64, lane, pk[cc]);
                }
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
#pragma unroll
                for (int cc = 0; cc < kChunks; cc += 2)
                    if (colbase + cc * 32 < p.N && row0 < p.M)
                        tma_store_3d(cc + 1 < kChunks ? map_w : map_d, colbase + cc * 32, row0, split, smem_u32(staging + cc * kStagingBytes));
                bulk_commit();
            }
        } else if (BUFS >= kChunks) {
            // a staging buffer per chunk: stage everything, make it visible once, then issue all the stores
            if (lane == 0) bulk_wait_read<0>();   // the stores of the previous tile have long been read
            __syncwarp();
#pragma unroll
            for (int cc = 0; cc < kChunks; cc++)
                if (colbase + cc * 32 < p.N && row0 < p.M) stage_line(staging + cc * kStagingBytes + lane * 64, lane, pk[cc]);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
#pragma unroll
                for (int cc = 0; cc < kChunks; cc++)
                    if (colbase + cc * 32 < p.N && row0 < p.M)
                        tma_store_3d(map_d, colbase + cc * 32, row0, split, smem_u32(staging + cc * kStagingBytes));
                bulk_commit();
            }
        } else {
#pragma unroll
            for (int cc = 0; cc < kChunks; cc++) {
                const int col = colbase + cc * 32;
                if (col < p.N && row0 < p.M) store_box(pk[cc], col);
            }
        }
    } else {
        // fp32 (dW and split-K partials: long K loops): chunk by chunk, 16 columns per box
#pragma unroll 1
        for (int cc = 0; cc < kChunks; cc++) {
            const int col = colbase + cc * 32;
            const bool live = col < p.N && row0 < p.M;
            uint32_t r[32];
            if (live) {
                tc_ld32(taddr + cc * 32, r);
                tc_wait_ld();
            }
            if (cc == kChunks - 1) release_acc();
            if (!live) continue;
            const int ncols = (int)min((int64_t)32, p.N - col);
            if (use_bias) {
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; j++) v[j] = __uint_as_float(r[j]);
                add_bias<32>(v, p.bias + col, ncols);
#pragma unroll
                for (int j = 0; j < 32; j++) r[j] = __float_as_uint(v[j]);
            }
            store_box(r, col);
            if (ncols > 16) store_box(r + 16, col + 16);
        }
    }
}

// ---- the roles that feed the tensor core (warps 0-3 of the single-CTA kernels) -------------------------------
// warp 0 / 3: TMA producers, warp 2: scale copier, warp 1: MMA issuer; C gives the shared-memory and TMEM layout.
template <class C, int BN>
__device__ __forceinline__ void gemm_feed_roles(int warp, uint32_t smem_base, uint32_t bar_full, uint32_t bar_sf_full, uint32_t bar_empty,
                                                uint32_t bar_acc_full, uint32_t bar_acc_empty, uint32_t tmem_base, volatile uint32_t *abort_flag,
                                                const CUtensorMap &map_a, const CUtensorMap &map_b, const GemmParams &p)
{
    const int items = p.tiles_m * p.tiles_n * p.splits;
    if (warp == 0 || warp == 3) {
        // ================= TMA producers =================
        // Issuing an asynchronous copy costs its thread on the order of 100 ns, and a stage needs five: warp 0 issues the
        // two operand tiles (and posts the byte count), warp 3 the scale chunks, both onto the stage's full barrier.
        {
            const bool leader = elect_one() && !p.withhold_loads;
            const bool operands = warp == 0;
            uint32_t stage = 0, phase = 0;
            bool alive = true;
            for (int item = blockIdx.x; item < items && alive; item += gridDim.x) {
                const int split = item % p.splits, tile = item / p.splits;
                const int mb = tile / p.tiles_n, nb = tile % p.tiles_n;
                const int kt0 = split * p.kt_per_split;
                const int kt1 = min(kt0 + p.kt_per_split, p.kt_total);
                // 128-row scale blocks of B that this tile touches (a 192-wide tile starts in the middle of one every other time)
                const int rb0 = (nb * BN) >> 7;
                int rbs = 0;
                for (int rb = 0; rb < C::kRB; rb++) rbs += (rb0 + rb) < p.rbB;
                for (int kt = kt0; kt < kt1; kt++) {
                    if (!mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                    const uint32_t sA = smem_base + stage * C::kStageBytes;
                    const uint32_t sB = sA + C::kABytes;
                    const uint32_t sSFA = sB + C::kBBytes;
                    const uint32_t sSFB = sSFA + C::kSfaBytes;
                    const uint32_t full = bar_full + 8 * stage;
                    // scale chunks present in this K tile (the last tile of an odd chunk count has one)
                    const int nch = min(2, p.nblk4 - 2 * kt);
                    if (leader && operands) {
                        mbar_expect_tx(full, (uint32_t)(C::kABytes + C::kBBytes + nch * kSfChunk * (1 + rbs)));
                        tma_load_2d(sA, &map_a, kt * kBKBytes, mb * kBM, full);
                        tma_load_2d(sB, &map_b, kt * kBKBytes, nb * BN, full);
                    }
                    if (leader && !operands) {
                        bulk_load(sSFA, p.sfa + ((size_t)mb * p.nblk4 + 2 * kt) * kSfChunk, (uint32_t)(nch * kSfChunk), full);
#pragma unroll
                        for (int rb = 0; rb < C::kRB; rb++)
                            if ((rb0 + rb) < p.rbB)
                                bulk_load(sSFB + rb * 2 * kSfChunk, p.sfb + ((size_t)(rb0 + rb) * p.nblk4 + 2 * kt) * kSfChunk,
                                          (uint32_t)(nch * kSfChunk), full);
                    }
                    __syncwarp();
                    if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 2) {
        // ================= scale copier =================
        // Stage s of the ring owns TMEM columns kSfCol + s * kSfSlot ..: they are free again exactly when the stage's
        // shared memory is (the producer refills it only after the MMAs that read both have completed).
        {
            const bool leader = elect_one();
            uint32_t stage = 0, phase = 0;
            bool alive = true;
            for (int item = blockIdx.x; item < items && alive; item += gridDim.x) {
                const int split = item % p.splits;
                const int kt0 = split * p.kt_per_split;
                const int kt1 = min(kt0 + p.kt_per_split, p.kt_total);
                for (int kt = kt0; kt < kt1; kt++) {
                    if (!mbar_wait_warp(bar_full + 8 * stage, phase, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t sSFA = smem_base + stage * C::kStageBytes + C::kABytes + C::kBBytes;
                    const uint32_t sSFB = sSFA + C::kSfaBytes;
                    const uint32_t t_sfa = tmem_base + C::kSfCol + stage * C::kSfSlot, t_sfb = t_sfa + 8;
                    const int64_t kleft = p.Kc - (int64_t)kt * kBKElems;
                    const int nch = kleft > 128 ? 2 : 1;
                    if (leader) {
#pragma unroll
                        for (int c = 0; c < 2; c++) {
                            if (c < nch) {
                                tc_cp_sf(t_sfa + 4 * c, desc_sf(sSFA + c * kSfChunk));
#pragma unroll
                                for (int rb = 0; rb < C::kRB; rb++)
                                    tc_cp_sf(t_sfb + 4 * C::kRB * c + 4 * rb, desc_sf(sSFB + rb * 2 * kSfChunk + c * kSfChunk));
                            }
                        }
                        tc_commit(bar_sf_full + 8 * stage);   // arrives once the copies have landed in TMEM
                    }
                    __syncwarp();
                    if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        // This warp's loop is the serial chain that bounds short and medium K loops (with every load, copy and store
        // taken out the kernel ran no faster), so it is kept short: one wait per stage (the scale copier has seen the
        // operands land before its copies, and its commit orders them before this warp's MMAs), and the barrier of the
        // NEXT stage is tested before this stage's MMAs are issued, so that the answer is there when it is needed.
        {
            const bool leader = elect_one();
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            const int nmma_last = (int)((p.Kc - (int64_t)(p.kt_total - 1) * kBKElems + 63) / 64);   // MMAs of the last K tile
            bool ready = false;   // the current stage's scales (hence operands) are known to be in place
            bool alive = true;
            for (int item = blockIdx.x; item < items && alive; item += gridDim.x) {
                const int split = item % p.splits, tile = item / p.splits;
                const int nb = tile % p.tiles_n;
                const int kt0 = split * p.kt_per_split;
                const int kt1 = min(kt0 + p.kt_per_split, p.kt_total);
                // scale columns hold 32 rows each: a tile that starts 64 rows into a 128-row block starts 2 columns in
                const uint32_t sfb_shift = (uint32_t)(((nb * BN) & 127) >> 5);
                if (!mbar_wait_warp(bar_acc_empty + 8 * acc, acc_phase ^ 1u, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kt = kt0; kt < kt1; kt++) {
                    if (!ready && !mbar_wait_warp(bar_sf_full + 8 * stage, phase, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t sA = smem_base + stage * C::kStageBytes;
                    const uint32_t sB = sA + C::kABytes;
                    const uint32_t t_sfa = tmem_base + C::kSfCol + stage * C::kSfSlot, t_sfb = t_sfa + 8 + sfb_shift;
                    const int nmma = kt == p.kt_total - 1 ? nmma_last : 4;
                    const uint64_t adesc = desc_operand_sw128(sA), bdesc = desc_operand_sw128(sB);
                    const uint32_t cur = stage;
                    if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
                    ready = __all_sync(0xFFFFFFFFu, mbar_test_wait(bar_sf_full + 8 * stage, phase));
                    if (leader) {
#pragma unroll
                        for (int k = 0; k < 4; k++) {
                            if (k < nmma) {
                                const uint32_t sf_id = (uint32_t)(k & 1) * 2u;
                                tc_mma_mxf4(d_tmem, adesc + (uint64_t)(k * (kMmaKBytes >> 4)), bdesc + (uint64_t)(k * (kMmaKBytes >> 4)),
                                            idesc_mxf4(BN, sf_id, sf_id), t_sfa + 4 * (k >> 1), t_sfb + 4 * C::kRB * (k >> 1),
                                            (kt > kt0 || k > 0) ? 1u : 0u);
                            }
                        }
                        tc_commit(bar_empty + 8 * cur);   // frees the stage (shared memory and scale columns) once these MMAs have read it
                    }
                }
                if (alive && leader) tc_commit(bar_acc_full + 8 * acc);  // accumulator complete
                __syncwarp();
                if (++acc == C::kAccStages) { acc = 0; acc_phase ^= 1u; }
            }
        }
    }
}

// ---- the kernel ------------------------------------------------------------------------------------
template <int BN, bool DEEP>
__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_mxf4(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const __grid_constant__ CUtensorMap map_d, const __grid_constant__ CUtensorMap map_dw, const GemmParams p)
{
    using C = GemmCfg<BN, DEEP>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + C::kBarOff);
    // barrier slots: full[kStages], sf_full[kStages], empty[kStages], acc_full[kAccStages], acc_empty[kAccStages]
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_sf_full = bar_full + 8 * C::kStages;
    const uint32_t bar_empty = bar_sf_full + 8 * C::kStages;
    const uint32_t bar_acc_full = bar_empty + 8 * C::kStages;
    const uint32_t bar_acc_empty = bar_acc_full + 8 * C::kAccStages;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 3 * C::kStages + 2 * C::kAccStages);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = smem_u32(smem);

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; s++) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_sf_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int a = 0; a < C::kAccStages; a++) {
            mbar_init(bar_acc_full + 8 * a, 1);
            mbar_init(bar_acc_empty + 8 * a, kEpiWarps);
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(C::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int items = p.tiles_m * p.tiles_n * p.splits;

    if (warp < kEpiWarp0) {
        gemm_feed_roles<C, BN>(warp, smem_base, bar_full, bar_sf_full, bar_empty, bar_acc_full, bar_acc_empty, tmem_base, abort_flag, map_a, map_b, p);
    } else if (warp >= kEpiWarp0) {
        // ================= epilogue (warps 4..11) =================
        const int ew = warp - kEpiWarp0;
        const int quarter = warp & 3;            // TMEM lanes 32*quarter .. +31 are the ones this warp may read
        const int chalf = ew >> 2;               // which half of the tile's columns this warp stores
        uint8_t *staging = smem + C::kStagingOff + ew * C::kStagingBufs * kStagingBytes;
        uint32_t sbuf = 0;                       // staging buffer of the next box (round robin)
        constexpr int kHalfCols = BN / 2;
        constexpr int kChunks = kHalfCols / 32;
        uint32_t acc = 0, acc_phase = 0;
        bool alive = true;
        for (int item = blockIdx.x; item < items && alive; item += gridDim.x) {
            const int split = item % p.splits, tile = item / p.splits;
            const int mb = tile / p.tiles_n, nb = tile % p.tiles_n;
            if (!mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
            tc_fence_after();
            const int row0 = mb * kBM + quarter * 32;
            const int colbase = nb * BN + chalf * kHalfCols;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN + chalf * kHalfCols;
            epilogue_tile<BN, C::kStagingBufs>(&map_d, p.out_fp32 ? nullptr : &map_dw, p, taddr, row0, colbase, split, staging, sbuf, lane,
                                               bar_acc_empty + 8 * acc);
            if (++acc == C::kAccStages) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) bulk_wait0();   // all stores of this warp have completed before the CTA may exit
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
    }
}

// ---- the quantizing kernel ------------------------------------------------------------------------------
// The product with the NEXT quantization fused into its epilogue (Sec. 3.3: every product's result is quantized again
// before the next product reads it).  Tiles are 128 x 128, exactly one tile of the two-axis quantizer: the epilogue
// warps cast their part of the accumulator (+ bias) to bf16 (Y), apply an elementwise hook (identity, GELU, or a
// multiplication by a caller's bf16 tensor: the derivative of an activation on the way back), round to bf16 again
// (Z) and lay Z down in shared memory in the layout the quantizer's passes read; Z can leave through TMA stores, Y
// through plain stores.  Then the same 256 threads run the row pass (codes of Z with groups along N, the forward /
// gradient operand of the next product) and the column pass (groups along M, stored transposed; with DQ it
// re-quantizes the dequantized result of the row pass: double quantization).  The results are bit for bit those of the
// stand-alone quantizers applied to Z.  Two accumulators: the next tile's K loop runs during this long epilogue.
template <bool WITH_Y>   // WITH_Y: a third tile for Y (stored beside a Z that differs from it) at the price of one ring stage
struct GemmQCfg {
    static constexpr int BN = 128;
    static constexpr int kRB = 1;
    static constexpr int kABytes = kBM * kBKBytes;
    static constexpr int kBBytes = BN * kBKBytes;
    static constexpr int kSfaBytes = 2 * kSfChunk;
    static constexpr int kSfbBytes = 2 * kSfChunk;
    static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;   // 34 KB
    static constexpr int kStages = WITH_Y ? 3 : 4;
    static constexpr int kAccStages = 2;
    static constexpr int kSfCol = kAccStages * BN;
    static constexpr int kSfSlot = 16;
    static constexpr int kTmemCols = 512;
    static constexpr int kTileOff = kStages * kStageBytes;           // Z, 32 KB
    static constexpr int kTile2Off = kTileOff + kTileBytes;          // DQ: dequantized row codes for the column pass; else: the hook's second factor
    static constexpr int kTileYOff = kTile2Off + kTileBytes;         // Y, when it is wanted beside a Z that differs from it
    static constexpr int kStagingOff = kTileYOff + (WITH_Y ? kTileBytes : 0);   // 2 x (transposed codes 8 KB + two scale chunks)
    static constexpr int kStagingBytes = kTile * 64 + 1024;
    static constexpr int kBarOff = kStagingOff + 2 * kStagingBytes;
    static constexpr int kSmemBytes = kBarOff + 1024 /*align*/ + 256 /*barriers*/;
    static_assert(kSfCol + kStages * kSfSlot <= 512, "TMEM budget");
    static_assert(kStageBytes % 1024 == 0 && kStagingBytes % 1024 == 0, "alignment");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

// GELU (0.5 y (1 + erf(y / sqrt 2))) in FP32.  erf by the rational form of Abramowitz & Stegun 7.1.26 (absolute error
// below 1.5e-7), one exponential and one reciprocal: the result is rounded to bf16, for which this is ample.
__device__ __forceinline__ float gelu_f32(float y)
{
    const float x = fabsf(y) * 0.70710678118654752f;
    float t, ex;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f, x, 1.0f)));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(ex) : "f"(x * x * -1.4426950408889634f));
    float poly = fmaf(1.061405429f, t, -1.453152027f);
    poly = fmaf(poly, t, 1.421413741f);
    poly = fmaf(poly, t, -0.284496736f);
    poly = fmaf(poly, t, 0.254829592f);
    const float erfc_abs = poly * t * ex;                         // 1 - erf(|y| / sqrt 2)
    const float half_y = 0.5f * y;
    // y >= 0: 0.5 y (2 - erfc) ; y < 0: 0.5 y erfc
    return half_y * (y >= 0.0f ? 2.0f - erfc_abs : erfc_abs);
}

struct QuantEpilogue {
    QuantSide rw, tr;             // row-wise result [M, N] and transposed result [N, M]
    int emit_row, emit_t;
    int hook;                     // MXFP4_HOOK_*
    const __nv_bfloat16 *aux;     // hook = multiply: bf16 [M, N]
    int64_t ld_aux;
    int store_y;                  // the bf16 result before the hook leaves through map_y
    int store_z;                  // the bf16 tile that is quantized leaves through map_z
    int aux_tma;                  // the hook's second factor arrives through map_aux (otherwise per-thread loads)
};

// named barrier of the 256 epilogue threads (barrier 0 belongs to __syncthreads)
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ bool epi_any(bool x)
{
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, 1, 256, q;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(r) : "r"((uint32_t)x) : "memory");
    return r != 0;
}

template <bool SR_ROW, bool SR_T, bool DQ, bool WITH_Y>
__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_mxf4_q(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
              const __grid_constant__ CUtensorMap map_y, const __grid_constant__ CUtensorMap map_z, const __grid_constant__ CUtensorMap map_aux,
              const __grid_constant__ CUtensorMap map_t, const GemmParams p, const __grid_constant__ QuantEpilogue e)
{
    using C = GemmQCfg<WITH_Y>;
    constexpr int BN = C::BN;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + C::kBarOff);
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_sf_full = bar_full + 8 * C::kStages;
    const uint32_t bar_empty = bar_sf_full + 8 * C::kStages;
    const uint32_t bar_acc_full = bar_empty + 8 * C::kStages;
    const uint32_t bar_acc_empty = bar_acc_full + 8 * C::kAccStages;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 3 * C::kStages + 2 * C::kAccStages);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    const uint32_t bar_aux = smem_u32(bars + 3 * C::kStages + 2 * C::kAccStages + 1);   // the hook's second factor has landed

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = smem_u32(smem);

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; s++) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_sf_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int a = 0; a < C::kAccStages; a++) {
            mbar_init(bar_acc_full + 8 * a, 1);
            mbar_init(bar_acc_empty + 8 * a, kEpiWarps);
        }
        mbar_init(bar_aux, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(C::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < kEpiWarp0) {
        gemm_feed_roles<C, BN>(warp, smem_base, bar_full, bar_sf_full, bar_empty, bar_acc_full, bar_acc_empty, tmem_base, abort_flag, map_a, map_b, p);
    } else {
        // ================= quantizing epilogue (warps 4..11 = 256 threads) =================
        const int et = (int)threadIdx.x - 32 * kEpiWarp0;
        const int quarter = warp & 3, chalf = (warp - kEpiWarp0) >> 2;
        const QsGeom g = qs_geom(et);
        const int M = (int)p.M, N = (int)p.N;
        const uint32_t tfa_r = tf_add_of(e.rw.scale_mode), tfa_t2 = tf_add_of(e.tr.scale_mode) * 0x00010001u;
        const uint32_t t_base = smem_base + C::kTileOff, t2_base = smem_base + C::kTile2Off, ty_base = smem_base + C::kTileYOff;
        const int trow = quarter * 32 + lane;                        // this thread's row of the tile
        const uint32_t row_off = (uint32_t)(chalf * (kTileBytes / 2) + trow * 128);
        const uint32_t t_row = t_base + row_off;
        // the hook's second factor travels by TMA into the second tile one tile ahead (that tile is free unless DQ uses it)
        const bool aux_tma = e.hook == MXFP4_HOOK_MULTIPLY && e.aux_tma && !DQ;
        auto issue_aux = [&](int item) {
            const int mb = item / p.tiles_n, nb = item % p.tiles_n;
            mbar_expect_tx(bar_aux, kTileBytes);
            tma_load_2d(t2_base, &map_aux, nb * BN, mb * kBM, bar_aux);
            tma_load_2d(t2_base + kTileBytes / 2, &map_aux, nb * BN + 64, mb * kBM, bar_aux);
        };
        if (aux_tma && et == 0 && !p.withhold_loads && (int)blockIdx.x < p.tiles_m * p.tiles_n) issue_aux(blockIdx.x);
        const bool use_bias = p.bias != nullptr;
        uint32_t nonfinite = 0;
        uint32_t acc = 0, acc_phase = 0;
        const int items = p.tiles_m * p.tiles_n;
        int it = 0;
        for (int item = blockIdx.x; item < items; item += gridDim.x, it++) {
            const int mb = item / p.tiles_n, nb = item % p.tiles_n;
            const int row0 = mb * kBM, col0 = nb * BN;
            bool ok = mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag, p.dev_status, p.spin_limit);
            if (aux_tma) ok = mbar_wait(bar_aux, (uint32_t)it & 1u, abort_flag, p.dev_status, p.spin_limit) && ok;
            if (epi_any(!ok)) break;      // a wait ran out in one of the eight warps: all of them leave together
            tc_fence_after();
            uint8_t *staging = smem + C::kStagingOff + (it & 1) * C::kStagingBytes;
            uint8_t *s_sc_row = staging + kTile * 64, *s_sc_t = s_sc_row + 512;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN + chalf * 64;
            const int grow = row0 + trow;

            // ---- accumulator -> Y (bf16) -> hook -> Z (bf16) -> the tile in shared memory ----
#pragma unroll
            for (int cc = 0; cc < 2; cc++) {
                const int col = col0 + chalf * 64 + cc * 32;
                const bool live = grow < M && col < N;     // N is a multiple of 32: a chunk is inside the matrix or outside it
                uint32_t r[32];
                tc_ld32(taddr + cc * 32, r);
                tc_wait_ld();
                if (cc == 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_acc_empty + 8 * acc);   // the accumulator goes back to the MMA issuer
                }
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; j++) v[j] = __uint_as_float(r[j]);
                if (use_bias && live) add_bias<32>(v, p.bias + col, 32);
                uint32_t yw[16];
#pragma unroll
                for (int j = 0; j < 16; j++) {
                    const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
                    yw[j] = *reinterpret_cast<const uint32_t *>(&h);
                }
                if (WITH_Y && e.store_y) {
#pragma unroll
                    for (int j = 0; j < 4; j++)
                        asm volatile("st.shared.v4.u32 [%4], {%0,%1,%2,%3};" ::"r"(yw[4 * j]), "r"(yw[4 * j + 1]), "r"(yw[4 * j + 2]), "r"(yw[4 * j + 3]),
                                     "r"(ty_base + row_off + (uint32_t)((((cc * 4 + j) ^ (trow & 7))) << 4)) : "memory");
                }
                uint32_t zw[16];
                if (e.hook == MXFP4_HOOK_GELU) {
#pragma unroll
                    for (int j = 0; j < 16; j++) {
                        const float a = bf16lo(yw[j]), b = bf16hi(yw[j]);
                        const __nv_bfloat162 h = __floats2bfloat162_rn(gelu_f32(a), gelu_f32(b));
                        zw[j] = *reinterpret_cast<const uint32_t *>(&h);
                    }
                } else if (e.hook == MXFP4_HOOK_MULTIPLY) {
                    uint4 aw[4] = {make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0)};
                    if (aux_tma) {
#pragma unroll
                        for (int j = 0; j < 4; j++)
                            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(aw[j].x), "=r"(aw[j].y), "=r"(aw[j].z), "=r"(aw[j].w)
                                         : "r"(t2_base + row_off + (uint32_t)((((cc * 4 + j) ^ (trow & 7))) << 4)));
                    } else if (live) {
                        const uint4 *ap = reinterpret_cast<const uint4 *>(e.aux + (int64_t)grow * e.ld_aux + col);
#pragma unroll
                        for (int j = 0; j < 4; j++) aw[j] = ld_nc_16(ap + j);
                    }
                    const uint32_t *a32 = reinterpret_cast<const uint32_t *>(aw);
#pragma unroll
                    for (int j = 0; j < 16; j++) {
                        // the product of two bf16 values is exact in FP32: one rounding, to bf16
                        const __nv_bfloat162 h = __floats2bfloat162_rn(bf16lo(yw[j]) * bf16lo(a32[j]), bf16hi(yw[j]) * bf16hi(a32[j]));
                        zw[j] = *reinterpret_cast<const uint32_t *>(&h);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 16; j++) zw[j] = yw[j];
                }
                if (!live) {
#pragma unroll
                    for (int j = 0; j < 16; j++) zw[j] = 0u;       // outside the matrix the tile holds zeros, as a TMA load would leave them
                }
#pragma unroll
                for (int j = 0; j < 4; j++)
                    asm volatile("st.shared.v4.u32 [%4], {%0,%1,%2,%3};" ::"r"(zw[4 * j]), "r"(zw[4 * j + 1]), "r"(zw[4 * j + 2]), "r"(zw[4 * j + 3]),
                                 "r"(t_row + (uint32_t)((((cc * 4 + j) ^ (trow & 7))) << 4)) : "memory");
            }
            fence_async_smem();
            epi_sync();                                   // the tile is complete, the second factor has been read
            if (et == 0) {
                if (e.store_z) {
                    tma_store_2d(&map_z, col0, row0, t_base);
                    tma_store_2d(&map_z, col0 + 64, row0, t_base + kTileBytes / 2);
                }
                if (WITH_Y && e.store_y) {
                    tma_store_2d(&map_y, col0, row0, ty_base);
                    tma_store_2d(&map_y, col0 + 64, row0, ty_base + kTileBytes / 2);
                }
                bulk_commit();
                if (aux_tma && item + (int)gridDim.x < items) issue_aux(item + gridDim.x);
            }
            if (e.emit_row) qs_row_pass<SR_ROW, DQ>(g, t_base, t2_base, row0, col0, M, N, e.rw, tfa_r, s_sc_row, nonfinite);
            if (DQ) __syncwarp();                         // the column pass reads what the row pass of the same warp wrote
            if (e.emit_t) qs_col_pass<SR_T>(g, DQ ? t2_base : t_base, row0, col0, M, N, e.tr, tfa_t2, staging, s_sc_t, nonfinite);
            fence_async_smem();
            if (et == 0) bulk_wait_read<0>();             // Z has left the tile, the previous tile's codes their staging buffer
            epi_sync();
            if (et == 0) {
                if (e.emit_t) {
                    tma_store_2d(&map_t, row0 >> 1, col0, smem_u32(staging));
                    bulk_store(e.tr.scales + ((size_t)(col0 >> 7) * e.tr.nblk4 + (row0 >> 7)) * 512, smem_u32(s_sc_t), 512);
                }
                if (e.emit_row) bulk_store(e.rw.scales + ((size_t)(row0 >> 7) * e.rw.nblk4 + (col0 >> 7)) * 512, smem_u32(s_sc_row), 512);
                bulk_commit();
            }
            if (++acc == C::kAccStages) { acc = 0; acc_phase ^= 1u; }
        }
        if (et == 0) bulk_wait0();
        if (nonfinite && p.dev_status) atomicOr(p.dev_status, MXFP4_DEV_NONFINITE);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
    }
}

// ---- the B-stationary kernel --------------------------------------------------------------------------
// For contraction lengths of a few K tiles (the forward and input-gradient products of the layers: Kc = 384 .. 1536)
// the ring of the kernel above carries, per stage, a B tile that the CTA has loaded many times before, and its rate
// is ring bytes in flight over load latency.  Here a CTA walks DOWN a column of tiles: the whole B block of the
// column (BN rows x Kc, with its scales in TMEM) stays resident, and the ring carries A alone, so that the same
// shared memory holds two to three times as many tiles in flight.  Tiles are numbered column by column and each CTA
// takes a contiguous range; B is reloaded where the range crosses into the next column.
template <int BN, int KT, int AS>   // KT: K tiles the resident B block can hold; AS: stages of the A ring
struct GemmBsCfg {
    static constexpr int kRB = (BN + 127) / 128;
    static constexpr int kABytes = kBM * kBKBytes;             // 16 KB
    static constexpr int kBBytes = BN * kBKBytes;              // one K tile of the B block
    static constexpr int kSfaBytes = 2 * kSfChunk;
    static constexpr int kSfbBytes = 2 * kSfChunk * kRB;       // per K tile
    static constexpr int kStagingBufs = (BN == 192 && KT > 2) ? 2 : BN / 64;
    static constexpr int kAOff = KT * kBBytes;
    static constexpr int kSfbOff = kAOff + AS * kABytes;
    static constexpr int kSfaOff = kSfbOff + KT * kSfbBytes;
    static constexpr int kStagingOff = kSfaOff + AS * kSfaBytes;
    static constexpr int kBarOff = kStagingOff + kEpiWarps * kStagingBufs * kStagingBytes;
    static constexpr int kSmemBytes = kBarOff + 1024 /*align*/ + 256 /*barriers*/;
    static constexpr int kSfbCol = 2 * BN;                     // TMEM columns: two accumulators, resident SFB (8 kRB per K tile), SFA ring (8 per stage)
    static constexpr int kSfaCol = kSfbCol + KT * 8 * kRB;
    static constexpr int kTmemCols = 512;
    static_assert(kSfaCol + AS * 8 <= 512, "TMEM budget");
    static_assert(kStagingOff % 1024 == 0, "staging alignment");
    static_assert(3 * AS + 7 <= 30, "barrier slots");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

template <int BN, int KT, int AS>
__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_mxf4_bs(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_d, const __grid_constant__ CUtensorMap map_dw, const GemmParams p)
{
    using C = GemmBsCfg<BN, KT, AS>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + C::kBarOff);
    // barrier slots: a_full[AS], sf_full[AS], a_empty[AS], acc_full[2], acc_empty[2], b_full, b_sf_full, b_empty
    const uint32_t bar_a_full = smem_u32(bars);
    const uint32_t bar_sf_full = bar_a_full + 8 * AS;
    const uint32_t bar_a_empty = bar_sf_full + 8 * AS;
    const uint32_t bar_acc_full = bar_a_empty + 8 * AS;
    const uint32_t bar_acc_empty = bar_acc_full + 16;
    const uint32_t bar_b_full = bar_acc_empty + 16;
    const uint32_t bar_b_sf_full = bar_b_full + 8;
    const uint32_t bar_b_empty = bar_b_sf_full + 8;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 3 * AS + 7);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = smem_u32(smem);

    if (threadIdx.x == 0) {
        for (int s = 0; s < AS; s++) {
            mbar_init(bar_a_full + 8 * s, 1);
            mbar_init(bar_sf_full + 8 * s, 1);
            mbar_init(bar_a_empty + 8 * s, 1);
        }
        for (int a = 0; a < 2; a++) {
            mbar_init(bar_acc_full + 8 * a, 1);
            mbar_init(bar_acc_empty + 8 * a, kEpiWarps);
        }
        mbar_init(bar_b_full, 1);
        mbar_init(bar_b_sf_full, 1);
        mbar_init(bar_b_empty, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(C::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // tiles are numbered column by column: t = nb * tiles_m + mb; this CTA owns [t0, t1)
    const int64_t total = (int64_t)p.tiles_m * p.tiles_n;
    const int t0 = (int)(total * blockIdx.x / gridDim.x), t1 = (int)(total * (blockIdx.x + 1) / gridDim.x);
    const int ktn = p.kt_total;

    if (warp == 0) {
        // ================= A producer: one A tile and its scales per stage =================
        const bool leader = elect_one() && !p.withhold_loads;
        uint32_t stage = 0, phase = 0;
        bool alive = true;
        for (int t = t0; t < t1 && alive; t++) {
            const int mb = t % p.tiles_m;
            for (int kt = 0; kt < ktn; kt++) {
                if (!mbar_wait_warp(bar_a_empty + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                const int nch = min(2, p.nblk4 - 2 * kt);
                if (leader) {
                    const uint32_t full = bar_a_full + 8 * stage;
                    mbar_expect_tx(full, (uint32_t)(C::kABytes + nch * kSfChunk));
                    tma_load_2d(smem_base + C::kAOff + stage * C::kABytes, &map_a, kt * kBKBytes, mb * kBM, full);
                    bulk_load(smem_base + C::kSfaOff + stage * C::kSfaBytes, p.sfa + ((size_t)mb * p.nblk4 + 2 * kt) * kSfChunk,
                              (uint32_t)(nch * kSfChunk), full);
                }
                __syncwarp();
                if (++stage == AS) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 3) {
        // ================= B producer: the block of a column, once per run of tiles in that column =================
        const bool leader = elect_one() && !p.withhold_loads;
        uint32_t runs = 0;
        for (int t = t0; t < t1;) {
            const int nb = t / p.tiles_m;
            // the MMAs of the previous column have finished reading the block
            if (runs > 0 && !mbar_wait_warp(bar_b_empty, (runs - 1u) & 1u, abort_flag, p.dev_status, p.spin_limit)) break;
            const int rb0 = (nb * BN) >> 7;
            int rbs = 0;
            for (int rb = 0; rb < C::kRB; rb++) rbs += (rb0 + rb) < p.rbB;
            if (leader) {
                mbar_expect_tx(bar_b_full, (uint32_t)(ktn * C::kBBytes + p.nblk4 * kSfChunk * rbs));
                for (int kt = 0; kt < ktn; kt++) {
                    const int nch = min(2, p.nblk4 - 2 * kt);
                    tma_load_2d(smem_base + kt * C::kBBytes, &map_b, kt * kBKBytes, nb * BN, bar_b_full);
#pragma unroll
                    for (int rb = 0; rb < C::kRB; rb++)
                        if ((rb0 + rb) < p.rbB)
                            bulk_load(smem_base + C::kSfbOff + kt * C::kSfbBytes + rb * 2 * kSfChunk,
                                      p.sfb + ((size_t)(rb0 + rb) * p.nblk4 + 2 * kt) * kSfChunk, (uint32_t)(nch * kSfChunk), bar_b_full);
                }
            }
            __syncwarp();
            runs++;
            t = min(t1, (nb + 1) * p.tiles_m);
        }
    } else if (warp == 2) {
        // ================= scale copier: B scales once per column, A scales per stage =================
        const bool leader = elect_one();
        uint32_t stage = 0, phase = 0, runs = 0;
        int cur_nb = -1;
        bool alive = true;
        for (int t = t0; t < t1 && alive; t++) {
            const int nb = t / p.tiles_m;
            if (nb != cur_nb) {
                if (!mbar_wait_warp(bar_b_full, runs & 1u, abort_flag, p.dev_status, p.spin_limit)) break;
                tc_fence_after();
                if (leader) {
                    for (int kt = 0; kt < ktn; kt++) {
                        const int nch = min(2, p.nblk4 - 2 * kt);
                        const uint32_t sSFB = smem_base + C::kSfbOff + kt * C::kSfbBytes;
                        const uint32_t t_sfb = tmem_base + C::kSfbCol + kt * 8 * C::kRB;
                        for (int c = 0; c < nch; c++)
#pragma unroll
                            for (int rb = 0; rb < C::kRB; rb++)
                                tc_cp_sf(t_sfb + 4 * C::kRB * c + 4 * rb, desc_sf(sSFB + rb * 2 * kSfChunk + c * kSfChunk));
                    }
                    tc_commit(bar_b_sf_full);
                }
                __syncwarp();
                cur_nb = nb;
                runs++;
            }
            for (int kt = 0; kt < ktn; kt++) {
                if (!mbar_wait_warp(bar_a_full + 8 * stage, phase, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                tc_fence_after();
                const uint32_t sSFA = smem_base + C::kSfaOff + stage * C::kSfaBytes;
                const uint32_t t_sfa = tmem_base + C::kSfaCol + stage * 8;
                const int nch = min(2, p.nblk4 - 2 * kt);
                if (leader) {
                    tc_cp_sf(t_sfa, desc_sf(sSFA));
                    if (nch > 1) tc_cp_sf(t_sfa + 4, desc_sf(sSFA + kSfChunk));
                    tc_commit(bar_sf_full + 8 * stage);   // arrives once the copies have landed in TMEM
                }
                __syncwarp();
                if (++stage == AS) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        const bool leader = elect_one();
        uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0, runs = 0;
        const int nmma_last = (int)((p.Kc - (int64_t)(ktn - 1) * kBKElems + 63) / 64);   // MMAs of the last K tile
        int cur_nb = -1;
        bool ready = false;
        bool alive = true;
        for (int t = t0; t < t1 && alive; t++) {
            const int nb = t / p.tiles_m;
            const bool last_of_run = (t + 1 == t1) || ((t + 1) / p.tiles_m != nb);
            if (nb != cur_nb) {
                // the block of this column and its scales are in place (the copier saw the block land before it copied)
                if (!mbar_wait_warp(bar_b_sf_full, runs & 1u, abort_flag, p.dev_status, p.spin_limit)) break;
                cur_nb = nb;
                runs++;
            }
            const uint32_t sfb_shift = (uint32_t)(((nb * BN) & 127) >> 5);
            if (!mbar_wait_warp(bar_acc_empty + 8 * acc, acc_phase ^ 1u, abort_flag, p.dev_status, p.spin_limit)) break;
            const uint32_t d_tmem = tmem_base + acc * BN;
            for (int kt = 0; kt < ktn; kt++) {
                if (!ready && !mbar_wait_warp(bar_sf_full + 8 * stage, phase, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                tc_fence_after();
                const uint64_t adesc = desc_operand_sw128(smem_base + C::kAOff + stage * C::kABytes);
                const uint64_t bdesc = desc_operand_sw128(smem_base + kt * C::kBBytes);
                const uint32_t t_sfa = tmem_base + C::kSfaCol + stage * 8;
                const uint32_t t_sfb = tmem_base + C::kSfbCol + kt * 8 * C::kRB + sfb_shift;
                const int nmma = kt == ktn - 1 ? nmma_last : 4;
                const uint32_t cur = stage;
                if (++stage == AS) { stage = 0; phase ^= 1u; }
                ready = __all_sync(0xFFFFFFFFu, mbar_test_wait(bar_sf_full + 8 * stage, phase));
                if (leader) {
#pragma unroll
                    for (int k = 0; k < 4; k++) {
                        if (k < nmma) {
                            const uint32_t sf_id = (uint32_t)(k & 1) * 2u;
                            tc_mma_mxf4(d_tmem, adesc + (uint64_t)(k * (kMmaKBytes >> 4)), bdesc + (uint64_t)(k * (kMmaKBytes >> 4)),
                                        idesc_mxf4(BN, sf_id, sf_id), t_sfa + 4 * (k >> 1), t_sfb + 4 * C::kRB * (k >> 1),
                                        (kt > 0 || k > 0) ? 1u : 0u);
                        }
                    }
                    tc_commit(bar_a_empty + 8 * cur);   // frees the A stage and its scale columns once these MMAs have read them
                }
            }
            if (alive && leader) {
                tc_commit(bar_acc_full + 8 * acc);            // accumulator complete
                if (last_of_run) tc_commit(bar_b_empty);      // and the resident block may be replaced
            }
            __syncwarp();
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    } else if (warp >= kEpiWarp0) {
        // ================= epilogue (warps 4..11) =================
        const int ew = warp - kEpiWarp0;
        const int quarter = warp & 3;
        const int chalf = ew >> 2;
        uint8_t *staging = smem + C::kStagingOff + ew * C::kStagingBufs * kStagingBytes;
        uint32_t sbuf = 0;
        constexpr int kHalfCols = BN / 2;
        uint32_t acc = 0, acc_phase = 0;
        for (int t = t0; t < t1; t++) {
            const int mb = t % p.tiles_m, nb = t / p.tiles_m;
            if (!mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag, p.dev_status, p.spin_limit)) break;
            tc_fence_after();
            const int row0 = mb * kBM + quarter * 32;
            const int colbase = nb * BN + chalf * kHalfCols;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN + chalf * kHalfCols;
            epilogue_tile<BN, C::kStagingBufs>(&map_d, p.out_fp32 ? nullptr : &map_dw, p, taddr, row0, colbase, 0, staging, sbuf, lane,
                                               bar_acc_empty + 8 * acc);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) bulk_wait0();   // all stores of this warp have completed before the CTA may exit
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
    }
}

// ---- the cluster split-K kernel -----------------------------------------------------------------------
// Weight-gradient products have a small output and a very long contraction: too few tiles for the machine.  Here the
// S CTAs of a thread-block cluster share ONE 128 x 192 tile, each taking 1/S of the contraction into its own
// accumulator, and the partial sums meet in distributed shared memory instead of in global memory: every CTA owns the
// 32-column chunks c with c mod S = its rank, receives those chunks from all S CTAs (its own included) into the shared
// memory its operand ring occupied, adds them in rank order (a fixed order: the result does not depend on timing)
// and stores the finished chunk.  No workspace, no second kernel.
//   barrier 1: every CTA's ring is idle (its MMAs have completed), so peers may write into it
//   barrier 2: all partial sums have arrived (release / acquire over the cluster)
// The tensor core adds into its FP32 accumulator with truncation, so the error of a sum grows with the number of MMAs
// chained into one accumulator.  A CTA here has a long chain (half of a long contraction), so it keeps TWO accumulators,
// one for its even and one for its odd K tiles, and adds them when it reads them out: the chains are as short as with
// four partial sums.
struct GemmCkCfg {
    static constexpr int BN = 192;
    static constexpr int kRB = 2;
    static constexpr int kABytes = kBM * kBKBytes;
    static constexpr int kBBytes = BN * kBKBytes;
    static constexpr int kSfaBytes = 2 * kSfChunk;
    static constexpr int kSfbBytes = 2 * kSfChunk * kRB;
    static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;   // 43 KB
    static constexpr int kStages = 5;
    static constexpr int kSfCol = 2 * BN;                               // TMEM: two accumulators (even / odd K tiles), then SFA (8) + SFB (16) per stage
    static constexpr int kSfSlot = 8 + 8 * kRB;
    static constexpr int kTmemCols = 512;
    static constexpr int kChunks = BN / 32;                             // 6: the cluster size divides it
    static constexpr int kChunkBytes = kBM * 32 * 4;                    // one 128 x 32 FP32 chunk: 16 KB
    static constexpr int kBarOff = kStages * kStageBytes;
    static constexpr int kSmemBytes = kBarOff + 1024 /*align*/ + 256 /*barriers*/;
    static_assert(kSfCol + kStages * kSfSlot <= 512, "TMEM budget");
    static_assert(kChunks * kChunkBytes <= kStages * kStageBytes, "the received chunks fit where the ring was");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

__device__ __forceinline__ uint32_t ck_cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t ck_cluster_size()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void ck_cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of `local` (a shared::cta address) in the shared memory of CTA `rank` of the cluster
__device__ __forceinline__ uint32_t ck_map(uint32_t local, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ void ck_store_remote(uint32_t addr, float a, float b, float c, float d)
{
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_mxf4_ck(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const GemmParams p)
{
    using C = GemmCkCfg;
    constexpr int BN = C::BN;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + C::kBarOff);
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_sf_full = bar_full + 8 * C::kStages;
    const uint32_t bar_empty = bar_sf_full + 8 * C::kStages;
    const uint32_t bar_acc_full = bar_empty + 8 * C::kStages;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 3 * C::kStages + 1);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t rank = ck_cluster_rank(), S = ck_cluster_size();

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; s++) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_sf_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_acc_full, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(C::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // the cluster's tile and this CTA's part of the contraction
    const int tile = (int)(blockIdx.x / S);
    const int mb = tile / p.tiles_n, nb = tile % p.tiles_n;
    const int kt0 = min((int)rank * p.kt_per_split, p.kt_total);
    const int kt1 = min(kt0 + p.kt_per_split, p.kt_total);
    const int rb0 = (nb * BN) >> 7;

    if (warp == 0 || warp == 3) {
        // ================= TMA producers (operands / scales) =================
        const bool leader = elect_one() && !p.withhold_loads;
        const bool operands = warp == 0;
        uint32_t stage = 0, phase = 0;
        int rbs = 0;
        for (int rb = 0; rb < C::kRB; rb++) rbs += (rb0 + rb) < p.rbB;
        for (int kt = kt0; kt < kt1; kt++) {
            if (!mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, p.spin_limit)) break;
            const uint32_t sA = smem_base + stage * C::kStageBytes;
            const uint32_t sB = sA + C::kABytes;
            const uint32_t sSFA = sB + C::kBBytes;
            const uint32_t sSFB = sSFA + C::kSfaBytes;
            const uint32_t full = bar_full + 8 * stage;
            const int nch = min(2, p.nblk4 - 2 * kt);
            if (leader && operands) {
                mbar_expect_tx(full, (uint32_t)(C::kABytes + C::kBBytes + nch * kSfChunk * (1 + rbs)));
                tma_load_2d(sA, &map_a, kt * kBKBytes, mb * kBM, full);
                tma_load_2d(sB, &map_b, kt * kBKBytes, nb * BN, full);
            }
            if (leader && !operands) {
                bulk_load(sSFA, p.sfa + ((size_t)mb * p.nblk4 + 2 * kt) * kSfChunk, (uint32_t)(nch * kSfChunk), full);
#pragma unroll
                for (int rb = 0; rb < C::kRB; rb++)
                    if ((rb0 + rb) < p.rbB)
                        bulk_load(sSFB + rb * 2 * kSfChunk, p.sfb + ((size_t)(rb0 + rb) * p.nblk4 + 2 * kt) * kSfChunk,
                                  (uint32_t)(nch * kSfChunk), full);
            }
            __syncwarp();
            if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
    } else if (warp == 2) {
        // ================= scale copier =================
        const bool leader = elect_one();
        uint32_t stage = 0, phase = 0;
        for (int kt = kt0; kt < kt1; kt++) {
            if (!mbar_wait_warp(bar_full + 8 * stage, phase, abort_flag, p.dev_status, p.spin_limit)) break;
            tc_fence_after();
            const uint32_t sSFA = smem_base + stage * C::kStageBytes + C::kABytes + C::kBBytes;
            const uint32_t sSFB = sSFA + C::kSfaBytes;
            const uint32_t t_sfa = tmem_base + C::kSfCol + stage * C::kSfSlot, t_sfb = t_sfa + 8;
            const int nch = min(2, p.nblk4 - 2 * kt);
            if (leader) {
#pragma unroll
                for (int c = 0; c < 2; c++) {
                    if (c < nch) {
                        tc_cp_sf(t_sfa + 4 * c, desc_sf(sSFA + c * kSfChunk));
#pragma unroll
                        for (int rb = 0; rb < C::kRB; rb++)
                            tc_cp_sf(t_sfb + 4 * C::kRB * c + 4 * rb, desc_sf(sSFB + rb * 2 * kSfChunk + c * kSfChunk));
                    }
                }
                tc_commit(bar_sf_full + 8 * stage);
            }
            __syncwarp();
            if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        const bool leader = elect_one();
        uint32_t stage = 0, phase = 0;
        const int nmma_last = (int)((p.Kc - (int64_t)(p.kt_total - 1) * kBKElems + 63) / 64);
        const uint32_t sfb_shift = (uint32_t)(((nb * BN) & 127) >> 5);
        bool alive = true;
        for (int kt = kt0; kt < kt1; kt++) {
            if (!mbar_wait_warp(bar_sf_full + 8 * stage, phase, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
            tc_fence_after();
            const uint32_t sA = smem_base + stage * C::kStageBytes;
            const uint64_t adesc = desc_operand_sw128(sA), bdesc = desc_operand_sw128(sA + C::kABytes);
            const uint32_t t_sfa = tmem_base + C::kSfCol + stage * C::kSfSlot, t_sfb = t_sfa + 8 + sfb_shift;
            const int nmma = kt == p.kt_total - 1 ? nmma_last : 4;
            if (leader) {
#pragma unroll
                for (int k = 0; k < 4; k++) {
                    if (k < nmma) {
                        const uint32_t sf_id = (uint32_t)(k & 1) * 2u;
                        tc_mma_mxf4(tmem_base + (uint32_t)((kt - kt0) & 1) * BN, adesc + (uint64_t)(k * (kMmaKBytes >> 4)),
                                    bdesc + (uint64_t)(k * (kMmaKBytes >> 4)), idesc_mxf4(BN, sf_id, sf_id), t_sfa + 4 * (k >> 1),
                                    t_sfb + 4 * C::kRB * (k >> 1), (kt - kt0 >= 2 || k > 0) ? 1u : 0u);
                    }
                }
                tc_commit(bar_empty + 8 * stage);
            }
            __syncwarp();
            if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
        if (alive && leader) tc_commit(bar_acc_full);   // also with no K tiles at all: nothing pending, arrives at once
        __syncwarp();
    }

    // ---- the epilogue warps wait for the accumulator; then the whole cluster meets: every ring is idle ----
    if (warp >= kEpiWarp0) {
        mbar_wait_warp(bar_acc_full, 0u, abort_flag, p.dev_status, p.spin_limit);
        tc_fence_after();
    }
    ck_cluster_sync();

    // ---- send: warp (quarter q, column half h) reads its 32 rows x 96 columns and hands each 32-column chunk to its owner ----
    const uint32_t slots = (uint32_t)((C::kChunks + S - 1) / S);    // chunks owned per CTA
    if (warp >= kEpiWarp0) {
        const int quarter = warp & 3, chalf = (warp - kEpiWarp0) >> 2;
        const int row = quarter * 32 + lane;
        const bool have = kt1 > kt0;          // a CTA without K tiles contributes zeros
        const bool have_odd = kt1 - kt0 >= 2; // the second accumulator has been written
#pragma unroll 1
        for (int cc = 0; cc < 3; cc++) {
            const uint32_t chunk = (uint32_t)(chalf * 3 + cc);
            uint32_t r[32];
            if (have) {
                tc_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + chunk * 32, r);
                tc_wait_ld();
                if (have_odd) {
                    uint32_t r2[32];
                    tc_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + BN + chunk * 32, r2);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; j++) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; j++) r[j] = 0u;
            }
            const uint32_t owner = chunk % S, slot = chunk / S;
            // receive area of the owner: [source rank][slot][row][32 floats], 16-byte pieces swizzled by the row
            const uint32_t local = smem_base + ((rank * slots + slot) * kBM + (uint32_t)row) * 128u;
            const uint32_t remote = ck_map(local, owner);
#pragma unroll
            for (int j = 0; j < 8; j++)
                ck_store_remote(remote + (uint32_t)((j ^ (row & 7)) << 4), __uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
        }
        tc_fence_before();
    }
    ck_cluster_sync();

    // ---- reduce and store the chunks this CTA owns: sources added in rank order ----
    {
        const bool use_bias = p.bias != nullptr;
        for (uint32_t slot = 0; slot < slots; slot++) {
            const uint32_t chunk = slot * S + rank;
            if (chunk >= (uint32_t)C::kChunks) break;
            const int col0 = nb * BN + (int)chunk * 32;
            if (col0 >= p.N) continue;
            for (int e = threadIdx.x; e < kBM * 8; e += kGemmThreads) {
                const int row = e >> 3, j = e & 7;
                const int grow = mb * kBM + row, gcol = col0 + j * 4;
                if (grow >= p.M || gcol >= p.N) continue;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (uint32_t src = 0; src < S; src++) {
                    const float4 v = *reinterpret_cast<const float4 *>(smem + ((src * slots + slot) * kBM + (uint32_t)row) * 128u +
                                                                        (uint32_t)((j ^ (row & 7)) << 4));
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
                if (use_bias) {
                    acc.x += __bfloat162float(p.bias[gcol]); acc.y += __bfloat162float(p.bias[gcol + 1]);
                    acc.z += __bfloat162float(p.bias[gcol + 2]); acc.w += __bfloat162float(p.bias[gcol + 3]);
                }
                if (p.out_fp32) {
                    *reinterpret_cast<float4 *>(static_cast<float *>(p.d) + (int64_t)grow * p.ldd + gcol) = acc;
                } else {
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
                    uint2 o;
                    o.x = *reinterpret_cast<const uint32_t *>(&lo);
                    o.y = *reinterpret_cast<const uint32_t *>(&hi);
                    *reinterpret_cast<uint2 *>(static_cast<__nv_bfloat16 *>(p.d) + (int64_t)grow * p.ldd + gcol) = o;
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
    }
}

// ---- MMA issue ceiling -----------------------------------------------------------------------------------
// What the tensor pipe takes when nothing else is in the way: one CTA per SM, operands and scales resident in shared
// memory / TMEM, one warp issuing kind::mxf4 MMAs of 128 x BN x 64 back to back into one accumulator, no loads, no
// scale copies inside the loop, no epilogue.  The rate of this loop is the ceiling a GEMM kernel on this part can be
// held against (the roofline denominators of the benchmark are measured copies and bf16 GEMMs, not FP4).
template <int BN>
__global__ void __launch_bounds__(128, 1) k_mma_ceiling(int iters, uint32_t *dev_status)
{
    constexpr int kRB = (BN + 127) / 128;
    constexpr int kABytes = kBM * kBKBytes, kBBytes = BN * kBKBytes, kSfBytes = 2 * kSfChunk * (1 + kRB);
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + kABytes + kBBytes + kSfBytes);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    const uint32_t smem_base = smem_u32(smem), bar_sf = smem_u32(bars), bar_done = bar_sf + 8;
    const int warp = threadIdx.x >> 5;

    // operands: any bit pattern is a valid pair of E2M1 codes; scales: 2^0
    for (int i = threadIdx.x; i < (kABytes + kBBytes) / 4; i += 128)
        reinterpret_cast<uint32_t *>(smem)[i] = 0x9E3779B9u * (uint32_t)(i + 1) + blockIdx.x;
    for (int i = threadIdx.x; i < kSfBytes / 4; i += 128) reinterpret_cast<uint32_t *>(smem + kABytes + kBBytes)[i] = 0x7F7F7F7Fu;
    if (threadIdx.x == 0) {
        mbar_init(bar_sf, 1);
        mbar_init(bar_done, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_async_smem();
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        const bool leader = elect_one();
        const uint32_t sSFA = smem_base + kABytes + kBBytes, sSFB = sSFA + 2 * kSfChunk;
        const uint32_t t_sfa = tmem_base + BN, t_sfb = t_sfa + 8;
        if (leader) {
#pragma unroll
            for (int c = 0; c < 2; c++) {
                tc_cp_sf(t_sfa + 4 * c, desc_sf(sSFA + c * kSfChunk));
#pragma unroll
                for (int rb = 0; rb < kRB; rb++) tc_cp_sf(t_sfb + 4 * kRB * c + 4 * rb, desc_sf(sSFB + rb * 2 * kSfChunk + c * kSfChunk));
            }
            tc_commit(bar_sf);
        }
        __syncwarp();
        bool ok = mbar_wait_warp(bar_sf, 0u, abort_flag, dev_status);
        tc_fence_after();
        const uint64_t adesc = desc_operand_sw128(smem_base), bdesc = desc_operand_sw128(smem_base + kABytes);
        for (int it = 0; it < iters && ok; it++) {
            if (leader) {
#pragma unroll
                for (int k = 0; k < 4; k++) {
                    const uint32_t sf_id = (uint32_t)(k & 1) * 2u;
                    tc_mma_mxf4(tmem_base, adesc + (uint64_t)(k * (kMmaKBytes >> 4)), bdesc + (uint64_t)(k * (kMmaKBytes >> 4)),
                                idesc_mxf4(BN, sf_id, sf_id), t_sfa + 4 * (k >> 1), t_sfb + 4 * kRB * (k >> 1), (it > 0 || k > 0) ? 1u : 0u);
                }
            }
            __syncwarp();
        }
        if (leader) tc_commit(bar_done);
        __syncwarp();
        mbar_wait_warp(bar_done, 0u, abort_flag, dev_status);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

// ---- the two-CTA kernel ---------------------------------------------------------------------------------
// A pair of CTAs (a cluster of two SMs) computes a 256 x 256 tile with tcgen05.mma.cta_group::2: each CTA holds 128
// rows of A, HALF of the B tile, the scales of its own A rows and the scales of all 256 B rows, and ends up with the
// accumulator of its own 128 rows.  Per SM and stage that is 32 KB of operands instead of 48 KB for the same flops:
// the single-CTA kernel is limited by operand delivery from L2, not by the tensor pipe.
// Roles per CTA are those of the single-CTA kernel, except that only the leader (rank 0) issues scale copies and MMAs
// (both act on the shared memory and TMEM of both CTAs), and warp 2 of the peer relays "my stage has landed" to the
// leader.  Stage and accumulator releases reach both CTAs through multicast commits.
template <bool DEEP>
struct Gemm2Cfg {
    static constexpr int kABytes = kBM * kBKBytes;                      // 16 KB: this CTA's 128 rows of A
    static constexpr int kBBytes = 128 * kBKBytes;                      // 16 KB: this CTA's half of the 256 B rows
    static constexpr int kSfaBytes = 2 * kSfChunk;
    static constexpr int kSfbBytes = 2 * kSfChunk * 2;                  // all 256 B rows
    static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;   // 35 KB
    // The loop is bound by operand bytes in flight over load latency, so every stage counts: six stages and a single
    // staging buffer per epilogue warp for long K loops (177 against 187 us at 8192^3), and no slack for aligning the
    // window: the kernel declares its window 1024-byte aligned and checks that it is.
    static constexpr int kStages = DEEP ? 4 : 6;
    static constexpr int kStagingBufs = DEEP ? 4 : 1;
    static constexpr int kSfCol = 256;                                  // TMEM: accumulator, then per ring stage SFA (8) + SFB (16)
    static constexpr int kSfSlot = 24;
    static constexpr int kTmemCols = 512;
    static constexpr int kStagingOff = kStages * kStageBytes;
    static constexpr int kBarOff = kStagingOff + kEpiWarps * kStagingBufs * kStagingBytes;
    static constexpr int kSmemBytes = kBarOff + 256 /*barriers*/;
    static_assert(kSfCol + kStages * kSfSlot <= 512, "TMEM budget");
    static_assert(kStageBytes % 1024 == 0 && kStagingOff % 1024 == 0, "alignment");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
// Non-blocking test: a suspended try_wait was seen to notice an arrival from the other CTA only after its time slice
// (about a microsecond), which stalls the pipeline every other stage.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait on a barrier that CTAs of the cluster arrive on; warp-uniform result.
__device__ __forceinline__ bool mbar_wait_cluster_warp(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *dev_status,
                                                       uint32_t limit)
{
    bool ok = false;
    for (uint32_t spin = 0; spin < limit; spin++) {
        if (mbar_try_wait_cluster(bar, parity)) { ok = true; break; }
        if (spin > 4096) {
            if (*abort_flag) break;
            __nanosleep(64);
        }
    }
    if (!ok && !*abort_flag) {
        *abort_flag = 1u;
        if (dev_status) atomicOr(dev_status, MXFP4_DEV_TIMEOUT);
    }
    return __all_sync(0xFFFFFFFFu, ok);
}
// Tile load whose completion is counted on a barrier that may live in the other CTA of the pair.
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar_cluster_addr)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes.cta_group::2 [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tc2_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc2_commit_both(uint32_t bar)   // the same barrier in both CTAs of the pair
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc2_cp_sf(uint32_t taddr, uint64_t sdesc)
{
    asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void tc2_mma_mxf4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t sfa_tmem,
                                             uint32_t sfb_tmem, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem) : "memory");
}
// Instruction descriptor of the pair MMA: M = 256 (128 rows per CTA), N = n (256 unless said otherwise).
__device__ __forceinline__ uint32_t idesc_mxf4_pair(uint32_t a_sf_id, uint32_t b_sf_id, int n = 256)
{
    return (b_sf_id << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | (1u << 23) | ((uint32_t)(256 >> 4) << 24) | (a_sf_id << 29);
}

template <bool DEEP>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
k_gemm_mxf4_pair(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_sfa, const __grid_constant__ CUtensorMap map_sfb,
                 const __grid_constant__ CUtensorMap map_d, const GemmParams p)
{
    using C = Gemm2Cfg<DEEP>;
    constexpr int BN = 256;
    extern __shared__ __align__(1024) uint8_t smem_aligned[];
    uint8_t *smem = smem_aligned;
    if (smem_u32(smem) & 1023u) {   // the swizzled operand tiles need it; nothing has been set up yet, so everybody just leaves
        if (threadIdx.x == 0 && p.dev_status) atomicOr(p.dev_status, MXFP4_DEV_SMEM_LAYOUT);
        return;
    }
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + C::kBarOff);
    // barrier slots: full[S] (used in the leader only: the loads of BOTH CTAs complete on it), sf_full[S], empty[S],
    // acc_full, acc_empty
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_sf_full = bar_full + 8 * C::kStages;
    const uint32_t bar_empty = bar_sf_full + 8 * C::kStages;
    const uint32_t bar_acc_full = bar_empty + 8 * C::kStages;
    const uint32_t bar_acc_empty = bar_acc_full + 8;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 4 * C::kStages + 2);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t rank = cluster_rank();

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; s++) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_sf_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_acc_full, 1);
        mbar_init(bar_acc_empty, 2 * kEpiWarps);   // the epilogue warps of both CTAs hand the accumulator back to the leader
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(C::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();     // both CTAs have their barriers and TMEM before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int tiles_m2 = (p.tiles_m + 1) >> 1;
    const int items = tiles_m2 * p.tiles_n * p.splits;
    const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;

    if (warp == 0 || warp == 3) {
        // ===== TMA producers (both CTAs: own rows of A and own half of B by warp 0; own SFA and all of SFB by warp 3) =====
        // All loads of both CTAs complete on the LEADER's full barrier (the cta_group::2 form of the load allows the
        // barrier to live in the other CTA of the pair), so the leader learns that a stage has landed in both shared
        // memories without any message between the CTAs.  The leader's warp 0 posts the byte count of both.
        const bool leader = elect_one() && !p.withhold_loads;
        const bool operands = warp == 0;
        uint32_t stage = 0, phase = 0;
        bool alive = true;
        for (int item = cluster_id; item < items && alive; item += num_clusters) {
            const int split = item % p.splits, tile = item / p.splits;
            const int mb = (tiles_m2 - 1 - tile / p.tiles_n) * 2 + (int)rank, nb = tile % p.tiles_n;
            const int kt0 = split * p.kt_per_split;
            const int kt1 = min(kt0 + p.kt_per_split, p.kt_total);
            for (int kt = kt0; kt < kt1; kt++) {
                if (!mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                const uint32_t sA = smem_base + stage * C::kStageBytes;
                const uint32_t sB = sA + C::kABytes;
                const uint32_t sSFA = sB + C::kBBytes;
                const uint32_t sSFB = sSFA + C::kSfaBytes;
                const uint32_t full = map_to_cta(bar_full + 8 * stage, 0);
                const int ktr = kt1 - 1 - (kt - kt0);   // the K tiles are taken from the last to the first
                if (leader && operands) {
                    if (rank == 0) mbar_expect_tx(bar_full + 8 * stage, 2u * (uint32_t)C::kStageBytes);
                    tma2_load_2d(sA, &map_a, ktr * kBKBytes, mb * kBM, full);
                    tma2_load_2d(sB, &map_b, ktr * kBKBytes, nb * BN + (int)rank * 128, full);
                }
                if (leader && !operands) {
                    // scale rows are 128-row blocks, 256 words (two 512-byte chunks) per stage; blocks beyond the matrix read as zero
                    tma2_load_2d(sSFA, &map_sfa, ktr * 256, mb, full);
                    tma2_load_2d(sSFB, &map_sfb, ktr * 256, nb * 2, full);
                }
                __syncwarp();
                if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 2) {
        // ================= scale copier (leader CTA only; each copy acts on both CTAs) =================
        if (rank == 0) {
            const bool leader = elect_one();
            uint32_t stage = 0, phase = 0;
            bool alive = true;
            for (int item = cluster_id; item < items && alive; item += num_clusters) {
                const int split = item % p.splits;
                const int kt0 = split * p.kt_per_split;
                const int kt1 = min(kt0 + p.kt_per_split, p.kt_total);
                for (int kt = kt0; kt < kt1; kt++) {
                    if (!mbar_wait_warp(bar_full + 8 * stage, phase, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t sSFA = smem_base + stage * C::kStageBytes + C::kABytes + C::kBBytes;
                    const uint32_t sSFB = sSFA + C::kSfaBytes;
                    const uint32_t t_sfa = tmem_base + C::kSfCol + stage * C::kSfSlot, t_sfb = t_sfa + 8;
                    const int64_t kleft = p.Kc - (int64_t)(kt1 - 1 - (kt - kt0)) * kBKElems;
                    const int nch = kleft > 128 ? 2 : 1;
                    if (leader) {
#pragma unroll
                        for (int c = 0; c < 2; c++) {
                            if (c < nch) {
                                tc2_cp_sf(t_sfa + 4 * c, desc_sf(sSFA + c * kSfChunk));
#pragma unroll
                                for (int rb = 0; rb < 2; rb++) tc2_cp_sf(t_sfb + 8 * c + 4 * rb, desc_sf(sSFB + rb * 2 * kSfChunk + c * kSfChunk));
                            }
                        }
                        tc2_commit(bar_sf_full + 8 * stage);   // arrives once the copies have landed in both TMEMs
                    }
                    __syncwarp();
                    if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer (leader CTA only) =================
        if (rank == 0) {
            const bool leader = elect_one();
            uint32_t stage = 0, phase = 0, acc_phase = 0;
            bool alive = true;
            for (int item = cluster_id; item < items && alive; item += num_clusters) {
                const int split = item % p.splits;
                const int kt0 = split * p.kt_per_split;
                const int kt1 = min(kt0 + p.kt_per_split, p.kt_total);
                if (!mbar_wait_cluster_warp(bar_acc_empty, acc_phase ^ 1u, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                tc_fence_after();
                for (int kt = kt0; kt < kt1; kt++) {
                    if (!mbar_wait_warp(bar_sf_full + 8 * stage, phase, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t sA = smem_base + stage * C::kStageBytes;
                    const uint32_t sB = sA + C::kABytes;
                    const uint32_t t_sfa = tmem_base + C::kSfCol + stage * C::kSfSlot, t_sfb = t_sfa + 8;
                    const int64_t kleft = p.Kc - (int64_t)(kt1 - 1 - (kt - kt0)) * kBKElems;
                    const int krem = kleft < kBKElems ? (int)kleft : kBKElems;
                    const int nmma = (krem + 63) / 64;
                    const uint64_t adesc = desc_operand_sw128(sA), bdesc = desc_operand_sw128(sB);
                    if (leader) {
#pragma unroll
                        for (int k = 0; k < 4; k++) {
                            if (k < nmma) {
                                const uint32_t sf_id = (uint32_t)(k & 1) * 2u;
                                tc2_mma_mxf4(tmem_base, adesc + (uint64_t)(k * (kMmaKBytes >> 4)), bdesc + (uint64_t)(k * (kMmaKBytes >> 4)),
                                             idesc_mxf4_pair(sf_id, sf_id), t_sfa + 4 * (k >> 1), t_sfb + 8 * (k >> 1),
                                             (kt > kt0 || k > 0) ? 1u : 0u);
                            }
                        }
                        tc2_commit_both(bar_empty + 8 * stage);   // frees the stage in both CTAs once these MMAs have read it
                    }
                    __syncwarp();
                    if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
                }
                if (alive && leader) tc2_commit_both(bar_acc_full);   // both CTAs' accumulators are complete
                __syncwarp();
                acc_phase ^= 1u;
            }
        }
    } else if (warp >= kEpiWarp0) {
        // ================= epilogue (warps 4..11 of both CTAs: own 128 rows x 256 columns) =================
        const int ew = warp - kEpiWarp0;
        const int quarter = warp & 3;
        const int chalf = ew >> 2;
        uint8_t *staging = smem + C::kStagingOff + ew * C::kStagingBufs * kStagingBytes;
        uint32_t sbuf = 0;
        constexpr int kHalfCols = BN / 2;
        constexpr int kChunks = kHalfCols / 32;
        const uint32_t acc_empty_leader = map_to_cta(bar_acc_empty, 0);
        uint32_t acc_phase = 0;
        bool alive = true;
        for (int item = cluster_id; item < items && alive; item += num_clusters) {
            const int split = item % p.splits, tile = item / p.splits;
            const int mb = (tiles_m2 - 1 - tile / p.tiles_n) * 2 + (int)rank, nb = tile % p.tiles_n;
            if (!mbar_wait_warp(bar_acc_full, acc_phase, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
            tc_fence_after();
            const int row0 = mb * kBM + quarter * 32;
            const int colbase = nb * BN + chalf * kHalfCols;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + chalf * kHalfCols;
            const bool use_bias = p.bias != nullptr && p.splits == 1;
            auto store_box = [&](const uint32_t *w, int x) {
                if (lane == 0) bulk_wait_read<C::kStagingBufs - 1>();
                __syncwarp();
                uint8_t *buf = staging + sbuf * kStagingBytes;
                stage_line(buf + lane * 64, lane, w);
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_3d(&map_d, x, row0, split, smem_u32(buf));
                    bulk_commit();
                }
                sbuf = (sbuf + 1) % C::kStagingBufs;
            };
            auto release_acc = [&]() {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_remote(acc_empty_leader);
            };
            if (!p.out_fp32) {
                uint32_t pk[kChunks][16];
#pragma unroll
                for (int cc = 0; cc < kChunks; cc++) {
                    const int col = colbase + cc * 32;
                    if (col < p.N && row0 < p.M) {
                        uint32_t r[32];
                        tc_ld32(taddr + cc * 32, r);
                        tc_wait_ld();
                        pack_row_bf16(r, use_bias ? p.bias + col : nullptr, (int)min((int64_t)32, p.N - col), pk[cc]);
                    }
                }
                release_acc();
                if (C::kStagingBufs >= kChunks) {
                    if (lane == 0) bulk_wait_read<0>();
                    __syncwarp();
#pragma unroll
                    for (int cc = 0; cc < kChunks; cc++)
                        if (colbase + cc * 32 < p.N && row0 < p.M) stage_line(staging + cc * kStagingBytes + lane * 64, lane, pk[cc]);
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
#pragma unroll
                        for (int cc = 0; cc < kChunks; cc++)
                            if (colbase + cc * 32 < p.N && row0 < p.M)
                                tma_store_3d(&map_d, colbase + cc * 32, row0, split, smem_u32(staging + cc * kStagingBytes));
                        bulk_commit();
                    }
                } else {
#pragma unroll
                    for (int cc = 0; cc < kChunks; cc++) {
                        const int col = colbase + cc * 32;
                        if (col < p.N && row0 < p.M) store_box(pk[cc], col);
                    }
                }
            } else {
#pragma unroll 1
                for (int cc = 0; cc < kChunks; cc++) {
                    const int col = colbase + cc * 32;
                    const bool live = col < p.N && row0 < p.M;
                    uint32_t r[32];
                    if (live) {
                        tc_ld32(taddr + cc * 32, r);
                        tc_wait_ld();
                    }
                    if (cc == kChunks - 1) release_acc();
                    if (!live) continue;
                    const int ncols = (int)min((int64_t)32, p.N - col);
                    if (use_bias) {
                        float v[32];
#pragma unroll
                        for (int j = 0; j < 32; j++) v[j] = __uint_as_float(r[j]);
                        add_bias<32>(v, p.bias + col, ncols);
#pragma unroll
                        for (int j = 0; j < 32; j++) r[j] = __float_as_uint(v[j]);
                    }
                    store_box(r, col);
                    if (ncols > 16) store_box(r + 16, col + 16);
                }
            }
            acc_phase ^= 1u;
        }
        if (lane == 0) bulk_wait0();
    }

    // neither CTA may leave (or free TMEM) while the other can still reach its shared memory, barriers or TMEM
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
    }
}

// ---- the two-CTA B-stationary kernel ----------------------------------------------------------------------
// Short contractions (Kc up to KT K tiles) with many rows: the forward and input-gradient products whose output write
// dominates.  The single-CTA kernels are bound there by shared-memory bandwidth (every operand byte is written once by
// TMA and read once by the tensor core through the same 128 B / cycle port) and the streaming pair kernel by its single
// accumulator.  Here a pair of CTAs walks DOWN a column of 256 x 192 tiles: each CTA keeps its half (96 rows) of the
// column's B block and the scales of all 192 B rows resident for the whole column, the ring carries this CTA's 128 rows
// of A alone (16 KB + 1 KB of scales per stage, eight stages), and two accumulators of 192 columns let the
// epilogue of one tile run under the K loop of the next.  Per stage and SM the port sees 16 KB written and 16 + 12 KB read for a 128 x 192 x 256
// block of the product, less than the tensor pipe needs for it.  Roles, barriers and the cross-CTA signalling are those
// of the two kernels this combines (k_gemm_mxf4_pair, k_gemm_mxf4_bs).
// The walk of one CTA pair over its range [t0, t1) of the column-by-column numbering.  Inside a column the pair does not
// take its rows in rising order but rotated so that it starts at a multiple of `period` (the range length, the same for
// every pair): all pairs then work on rows of the same residue at the same time, i.e. the pairs that need an A tile (one
// per column) ask for it within a few microseconds of one another instead of spread over the whole kernel, and it comes
// from L2 (in rising order an A tile of 50432 x 4096 x 1024 was read from DRAM about four times; 116 -> 109 us).  The
// single-CTA B-stationary kernel (short contractions, small A operands) gains nothing from the same walk.
struct PbsWalk {
    int tiles_m2, t0, t1, period;
};
struct PbsTile {
    int nb, mb2;
    bool first, last;   // of this pair's run in the column nb
};
__device__ __forceinline__ PbsTile pbs_tile(const PbsWalk &w, int t)
{
    PbsTile x;
    x.nb = t / w.tiles_m2;
    const int c0 = x.nb * w.tiles_m2;
    const int lo = max(w.t0, c0), hi = min(w.t1, c0 + w.tiles_m2);   // this pair's run in the column
    const int len = hi - lo, ra = lo - c0;
    const int s = ((ra + w.period - 1) / w.period) * w.period;         // first multiple of the period at or after the run's first row
    const int rot = s < ra + len ? s - ra : 0;
    int o = t - lo + rot;
    if (o >= len) o -= len;
    x.mb2 = ra + o;
    x.first = t == lo;
    x.last = t == hi - 1;
    return x;
}

template <int KT, int AS>   // KT: K tiles the resident B block can hold; AS: stages of the A ring
struct GemmPbsCfg {
    static constexpr int BN = 192;
    static constexpr int kABytes = kBM * kBKBytes;              // 16 KB: this CTA's 128 rows of A
    static constexpr int kBBytes = (BN / 2) * kBKBytes;         // 12 KB: this CTA's 96 B rows of one K tile
    static constexpr int kSfaBytes = 2 * kSfChunk;
    static constexpr int kSfbBytes = 2 * kSfChunk * 2;          // per K tile: the two 128-row blocks a tile touches
    static constexpr int kStagingBufs = 2;                     // the ring is worth more than a third buffer: the loop is bound by operand bytes in flight
    static constexpr int kAOff = KT * kBBytes;
    static constexpr int kSfbOff = kAOff + AS * kABytes;
    static constexpr int kSfaOff = kSfbOff + KT * kSfbBytes;
    static constexpr int kStagingOff = kSfaOff + AS * kSfaBytes;
    static constexpr int kBarOff = kStagingOff + kEpiWarps * kStagingBufs * kStagingBytes;
    static constexpr int kSmemBytes = kBarOff + 1024 /*align*/ + 512 /*barriers*/;
    static constexpr int kSfbCol = 2 * BN;                      // TMEM columns: two accumulators, resident SFB (16 per K tile), SFA ring (8 per stage)
    static constexpr int kSfaCol = kSfbCol + KT * 16;
    static constexpr int kTmemCols = 512;
    static_assert(kSfaCol + AS * 8 <= 512, "TMEM budget");
    static_assert(kAOff % 1024 == 0 && kStagingOff % 1024 == 0, "alignment");
    static_assert((3 * AS + 7) * 8 + 8 <= 512, "barrier slots");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

template <int KT, int AS>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
k_gemm_mxf4_pbs(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                const __grid_constant__ CUtensorMap map_sfa, const __grid_constant__ CUtensorMap map_sfb,
                const __grid_constant__ CUtensorMap map_d, const __grid_constant__ CUtensorMap map_dw, const GemmParams p)
{
    using C = GemmPbsCfg<KT, AS>;
    constexpr int BN = C::BN;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + C::kBarOff);
    // barrier slots: a_full[AS] and b_full (used in the leader only: the loads of BOTH CTAs complete on them), sf_full[AS],
    // b_sf_full (leader only), a_empty[AS], b_empty, acc_full[2] (both CTAs, through multicast commits), acc_empty[2] (leader)
    const uint32_t bar_a_full = smem_u32(bars);
    const uint32_t bar_sf_full = bar_a_full + 8 * AS;
    const uint32_t bar_a_empty = bar_sf_full + 8 * AS;
    const uint32_t bar_acc_full = bar_a_empty + 8 * AS;
    const uint32_t bar_acc_empty = bar_acc_full + 16;
    const uint32_t bar_b_full = bar_acc_empty + 16;
    const uint32_t bar_b_sf_full = bar_b_full + 8;
    const uint32_t bar_b_empty = bar_b_sf_full + 8;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 3 * AS + 7);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t rank = cluster_rank();

    if (threadIdx.x == 0) {
        for (int s = 0; s < AS; s++) {
            mbar_init(bar_a_full + 8 * s, 1);
            mbar_init(bar_sf_full + 8 * s, 1);
            mbar_init(bar_a_empty + 8 * s, 1);
        }
        for (int a = 0; a < 2; a++) {
            mbar_init(bar_acc_full + 8 * a, 1);
            mbar_init(bar_acc_empty + 8 * a, 2 * kEpiWarps);   // the epilogue warps of both CTAs hand an accumulator back to the leader
        }
        mbar_init(bar_b_full, 1);
        mbar_init(bar_b_sf_full, 1);
        mbar_init(bar_b_empty, 2);    // both MMA issuers
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(C::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();     // both CTAs have their barriers and TMEM before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // pair tiles (256 rows x 192 columns) are numbered column by column: t = nb * tiles_m2 + mb2; this pair owns [t0, t1)
    // and walks it as pbs_tile says
    const int tiles_m2 = (p.tiles_m + 1) >> 1;
    const int64_t total = (int64_t)tiles_m2 * p.tiles_n;
    const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
    const int t0 = (int)(total * cluster_id / num_clusters), t1 = (int)(total * (cluster_id + 1) / num_clusters);
    const int ktn = p.kt_total;
    const PbsWalk walk = {tiles_m2, t0, t1, max(1, (int)((total + num_clusters - 1) / num_clusters))};

    if (warp == 0) {
        // ===== producer (both CTAs): own 128 rows of A and their scales per stage; own half of a column's B block and all
        // its scales once per run of tiles in that column.  Everything is counted on the LEADER's barriers. =====
        const bool leader = elect_one() && !p.withhold_loads;
        uint32_t stage = 0, phase = 0, runs = 0;
        int nb = 0;
        bool alive = true;
        auto load_block = [&]() -> bool {
            // the MMAs of the previous column have finished reading the block (multicast commits reach both CTAs)
            if (runs > 0 && !mbar_wait_warp(bar_b_empty, (runs - 1u) & 1u, abort_flag, p.dev_status, p.spin_limit)) return false;
            if (leader) {
                const uint32_t full = map_to_cta(bar_b_full, 0);
                if (rank == 0) mbar_expect_tx(bar_b_full, 2u * (uint32_t)ktn * (uint32_t)(C::kBBytes + C::kSfbBytes));
                for (int kt = 0; kt < ktn; kt++) {
                    tma2_load_2d(smem_base + kt * C::kBBytes, &map_b, kt * kBKBytes, nb * BN + (int)rank * (BN / 2), full);
                    // scale rows are 128-row blocks, 256 words (two 512-byte chunks) per K tile; what lies beyond the matrix reads as zero
                    tma2_load_2d(smem_base + C::kSfbOff + kt * C::kSfbBytes, &map_sfb, kt * 256, (nb * BN) >> 7, full);
                }
            }
            __syncwarp();
            runs++;
            return true;
        };
        for (int t = t0; t < t1 && alive; t++) {
            // the first block before anything else; later ones after the A stages of the column's first tile, which need
            // nothing from the new block and keep the ring full while the old column drains
            const PbsTile x = pbs_tile(walk, t);
            nb = x.nb;
            if (t == t0 && !load_block()) break;
            const int mb = x.mb2 * 2 + (int)rank;
            for (int kt = 0; kt < ktn; kt++) {
                if (!mbar_wait_warp(bar_a_empty + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                if (leader) {
                    const uint32_t full = map_to_cta(bar_a_full + 8 * stage, 0);
                    if (rank == 0) mbar_expect_tx(bar_a_full + 8 * stage, 2u * (uint32_t)(C::kABytes + C::kSfaBytes));
                    tma2_load_2d(smem_base + C::kAOff + stage * C::kABytes, &map_a, kt * kBKBytes, mb * kBM, full);
                    tma2_load_2d(smem_base + C::kSfaOff + stage * C::kSfaBytes, &map_sfa, kt * 256, mb, full);
                }
                __syncwarp();
                if (++stage == AS) { stage = 0; phase ^= 1u; }
            }
            if (alive && t != t0 && x.first && !load_block()) break;
        }
    } else if (warp == 2) {
        // ===== scale copier (leader only; each copy acts on both CTAs): B scales once per column, A scales per stage =====
        if (rank == 0) {
            const bool leader = elect_one();
            uint32_t stage = 0, phase = 0, runs = 0;
            bool alive = true;
            for (int t = t0; t < t1 && alive; t++) {
                if (pbs_tile(walk, t).first) {
                    if (!mbar_wait_warp(bar_b_full, runs & 1u, abort_flag, p.dev_status, p.spin_limit)) break;
                    tc_fence_after();
                    if (leader) {
                        for (int kt = 0; kt < ktn; kt++) {
                            const int nch = min(2, p.nblk4 - 2 * kt);
                            const uint32_t sSFB = smem_base + C::kSfbOff + kt * C::kSfbBytes;
                            const uint32_t t_sfb = tmem_base + C::kSfbCol + kt * 16;
                            for (int c = 0; c < nch; c++)
#pragma unroll
                                for (int rb = 0; rb < 2; rb++) tc2_cp_sf(t_sfb + 8 * c + 4 * rb, desc_sf(sSFB + rb * 2 * kSfChunk + c * kSfChunk));
                        }
                        tc2_commit(bar_b_sf_full);
                    }
                    __syncwarp();
                    runs++;
                }
                for (int kt = 0; kt < ktn; kt++) {
                    if (!mbar_wait_warp(bar_a_full + 8 * stage, phase, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t sSFA = smem_base + C::kSfaOff + stage * C::kSfaBytes;
                    const uint32_t t_sfa = tmem_base + C::kSfaCol + stage * 8;
                    const int nch = min(2, p.nblk4 - 2 * kt);
                    if (leader) {
                        tc2_cp_sf(t_sfa, desc_sf(sSFA));
                        if (nch > 1) tc2_cp_sf(t_sfa + 4, desc_sf(sSFA + kSfChunk));
                        tc2_commit(bar_sf_full + 8 * stage);   // arrives once the copies have landed in both TMEMs
                    }
                    __syncwarp();
                    if (++stage == AS) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1 || warp == 3) {
        // ===== MMA issuers (leader only): warp 1 takes this pair's even tiles into accumulator 0, warp 3 the odd ones
        // into accumulator 1.  One issuing thread needs about 350 cycles per stage (a barrier query, four MMAs, a commit)
        // and several hundred per tile, more than the tensor pipe needs for the stage; two of them leave it waiting for
        // nothing but operands.  Both walk over EVERY stage and every column in order and wait on each barrier phase
        // (a wait that skipped a phase could mistake the phase before for the one it wants); a warp issues and commits only
        // for its own tiles, so a stage's release tracks exactly the MMAs that read it (commits count the issuing thread's
        // operations), and the resident block is released by both (its barrier counts two arrivals). =====
        if (rank == 0) {
            const bool leader = elect_one();
            const uint32_t me = warp == 1 ? 0u : 1u;
            uint32_t stage = 0, phase = 0, acc_phase = 0, runs = 0;
            const int nmma_last = (int)((p.Kc - (int64_t)(ktn - 1) * kBKElems + 63) / 64);   // MMAs of the last K tile
            const uint32_t d_tmem = tmem_base + me * BN;
            bool alive = true;
            for (int t = t0; t < t1 && alive; t++) {
                const bool mine = (uint32_t)((t - t0) & 1) == me;
                const PbsTile x = pbs_tile(walk, t);
                const int nb = x.nb;
                const bool last_of_run = x.last;
                if (x.first) {
                    // the block of this column and its scales are in place in both CTAs (the copier saw them land before it copied)
                    if (!mbar_wait_warp(bar_b_sf_full, runs & 1u, abort_flag, p.dev_status, p.spin_limit)) break;
                    runs++;
                }
                // scale columns hold 32 rows each: a tile that starts 64 rows into a 128-row block starts 2 columns in
                const uint32_t sfb_shift = (uint32_t)(((nb * BN) & 127) >> 5);
                if (mine) {
                    if (!mbar_wait_cluster_warp(bar_acc_empty + 8 * me, acc_phase ^ 1u, abort_flag, p.dev_status, p.spin_limit)) break;
                    acc_phase ^= 1u;
                }
                for (int kt = 0; kt < ktn; kt++) {
                    if (!mbar_wait_warp(bar_sf_full + 8 * stage, phase, abort_flag, p.dev_status, p.spin_limit)) { alive = false; break; }
                    if (mine) {
                        tc_fence_after();
                        const uint64_t adesc = desc_operand_sw128(smem_base + C::kAOff + stage * C::kABytes);
                        const uint64_t bdesc = desc_operand_sw128(smem_base + kt * C::kBBytes);
                        const uint32_t t_sfa = tmem_base + C::kSfaCol + stage * 8;
                        const uint32_t t_sfb = tmem_base + C::kSfbCol + kt * 16 + sfb_shift;
                        const int nmma = kt == ktn - 1 ? nmma_last : 4;
                        if (leader) {
#pragma unroll
                            for (int k = 0; k < 4; k++) {
                                if (k < nmma) {
                                    const uint32_t sf_id = (uint32_t)(k & 1) * 2u;
                                    tc2_mma_mxf4(d_tmem, adesc + (uint64_t)(k * (kMmaKBytes >> 4)), bdesc + (uint64_t)(k * (kMmaKBytes >> 4)),
                                                 idesc_mxf4_pair(sf_id, sf_id, BN), t_sfa + 4 * (k >> 1), t_sfb + 8 * (k >> 1),
                                                 (kt > 0 || k > 0) ? 1u : 0u);
                                }
                            }
                            tc2_commit_both(bar_a_empty + 8 * stage);   // frees the A stage in both CTAs once these MMAs have read it
                        }
                        __syncwarp();
                    }
                    if (++stage == AS) { stage = 0; phase ^= 1u; }
                }
                if (alive && leader) {
                    if (mine) tc2_commit_both(bar_acc_full + 8 * me);   // both CTAs' accumulators are complete
                    if (last_of_run) tc2_commit_both(bar_b_empty);      // this warp's MMAs on the resident blocks are complete
                }
                __syncwarp();
            }
        }
    } else if (warp >= kEpiWarp0) {
        // ===== epilogue (warps 4..11 of both CTAs: own 128 rows x 192 columns) =====
        const int ew = warp - kEpiWarp0;
        const int quarter = warp & 3;
        const int chalf = ew >> 2;
        uint8_t *staging = smem + C::kStagingOff + ew * C::kStagingBufs * kStagingBytes;
        uint32_t sbuf = 0;
        constexpr int kHalfCols = BN / 2;
        uint32_t acc = 0, acc_phase = 0;
        for (int t = t0; t < t1; t++) {
            const PbsTile x = pbs_tile(walk, t);
            const int mb = x.mb2 * 2 + (int)rank, nb = x.nb;
            if (!mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag, p.dev_status, p.spin_limit)) break;
            tc_fence_after();
            const int row0 = mb * kBM + quarter * 32;
            const int colbase = nb * BN + chalf * kHalfCols;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN + chalf * kHalfCols;
            epilogue_tile<BN, C::kStagingBufs, true>(&map_d, p.out_fp32 ? nullptr : &map_dw, p, taddr, row0, colbase, 0, staging, sbuf, lane,
                                                     map_to_cta(bar_acc_empty + 8 * acc, 0));
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) bulk_wait0();   // all stores of this warp have completed before the CTA may exit
    }

    // neither CTA may leave (or free TMEM) while the other can still reach its shared memory, barriers or TMEM
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
    }
}

// Split-K: sum the FP32 partials in a fixed order, add the bias, cast.
__global__ void __launch_bounds__(256) k_splitk_reduce(const float *__restrict__ part, int splits, int64_t M, int64_t N,
                                                       void *__restrict__ d, int64_t ldd, int out_fp32,
                                                       const __nv_bfloat16 *__restrict__ bias)
{
    const int64_t total4 = M * N / 4;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total4; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t e = i * 4, row = e / N, col = e - row * N;
        float4 acc = *reinterpret_cast<const float4 *>(part + e);
        for (int s = 1; s < splits; s++) {
            const float4 v = *reinterpret_cast<const float4 *>(part + (size_t)s * M * N + e);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        if (bias) {
            acc.x += __bfloat162float(bias[col]); acc.y += __bfloat162float(bias[col + 1]);
            acc.z += __bfloat162float(bias[col + 2]); acc.w += __bfloat162float(bias[col + 3]);
        }
        if (out_fp32) {
            *reinterpret_cast<float4 *>(static_cast<float *>(d) + row * ldd + col) = acc;
        } else {
            __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
            uint2 o;
            o.x = *reinterpret_cast<uint32_t *>(&lo);
            o.y = *reinterpret_cast<uint32_t *>(&hi);
            *reinterpret_cast<uint2 *>(static_cast<__nv_bfloat16 *>(d) + row * ldd + col) = o;
        }
    }
}

// ---- host side -------------------------------------------------------------------------------------
// Packed operand [rows, kc/2 bytes] viewed as a 2-D byte tensor; box = 128 bytes x box_rows, 128B swizzle.
static bool make_operand_map(CUtensorMap *map, const void *data, int64_t rows, int64_t kc, int box_rows)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)(kc / 2), (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)(kc / 2)};
    cuuint32_t box[2] = {(cuuint32_t)kBKBytes, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return encode_tiled_cached(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(data), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Scales of a packed [rows, kc] matrix as a 2-D tensor of 32-bit words: one row per 128-row block, 128 words per
// 512-byte chunk; box = 256 words (the two chunks of a 256-K stage) x box_blocks, no swizzle, zero beyond the edges.
static bool make_scale_map(CUtensorMap *map, const void *scales, int64_t rows, int64_t kc, int box_blocks)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const cuuint64_t nblk4 = (cuuint64_t)ceil_div(kc / 32, 4);
    cuuint64_t gdim[2] = {nblk4 * 128, (cuuint64_t)ceil_div(rows, 128)};
    cuuint64_t gstride[1] = {nblk4 * 512};
    cuuint32_t box[2] = {256, (cuuint32_t)box_blocks};
    cuuint32_t estr[2] = {1, 1};
    return encode_tiled_cached(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void *>(scales), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Output [splits][M][N] (splits = 1: the caller's matrix with leading dimension ld) as a 3-D tensor for the
// epilogue's stores; box = 64 bytes x 32 rows, 64B swizzle.  Stores are clipped at M and N.
static bool make_output_map(CUtensorMap *map, void *d, int64_t m, int64_t n, int64_t ld, int splits, bool fp32)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const cuuint64_t esz = fp32 ? 4 : 2;
    cuuint64_t gdim[3] = {(cuuint64_t)n, (cuuint64_t)m, (cuuint64_t)splits};
    cuuint64_t gstride[2] = {(cuuint64_t)ld * esz, (cuuint64_t)m * (cuuint64_t)ld * esz};
    cuuint32_t box[3] = {(cuuint32_t)(64 / esz), 32, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return encode_tiled_cached(map, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, d, gdim, gstride, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The bf16 output once more with boxes of 64 columns x 32 rows and 128B swizzle (pairs of 32-column chunks in one store).
static bool make_output_map_wide(CUtensorMap *map, void *d, int64_t m, int64_t n, int64_t ld)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[3] = {(cuuint64_t)n, (cuuint64_t)m, 1};
    cuuint64_t gstride[2] = {(cuuint64_t)ld * 2, (cuuint64_t)m * (cuuint64_t)ld * 2};
    cuuint32_t box[3] = {64, 32, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return encode_tiled_cached(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, d, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct GemmPlan {
    bool deep;   // short K loop per tile: favour the epilogue (more staging, shorter ring)
    bool pair;   // 256 x 256 tiles on pairs of CTAs (cta_group::2)
    int bs;      // B-stationary kernel: 0 = no, 1 = 192 wide, up to 2 K tiles
    int ck;      // cluster split-K kernel: 0 = no, else the cluster size (CTAs sharing one 128 x 192 tile)
    bool pbs;    // two-CTA B-stationary kernel: 256 x 192 tiles, up to 4 K tiles
    int bn, tiles_m, tiles_n, splits, kt_total, kt_per_split;
};

// Tile width, CTA pairing and split-K factor.
// An MMA takes the same time for any width up to 256, so wide tiles are cheaper per flop; but only tiles up to 192
// wide leave room in TMEM for a second accumulator, which hides the epilogue behind the next K loop.  For long K
// loops the product is limited by operand delivery from L2, and pairs of CTAs sharing the B tile cut that by a third.
// Split K when the output has too few tiles to fill the machine.
static GemmPlan plan_gemm(int64_t m, int64_t n, int64_t kc, int sms, bool allow_split = true)
{
    GemmPlan g;
    g.kt_total = (int)ceil_div(kc, kBKElems);
    g.bs = 0;
    g.ck = 0;
    g.pbs = false;
    if (g.kt_total >= 16) {
        // Few tiles, long contraction (weight-gradient products): pairs of CTAs share a 128 x 192 tile and add their
        // halves of the contraction through distributed shared memory, when that fills between half and all of the
        // machine.  Larger clusters lose: a cluster of six such CTAs (a whole SM each) finds room only 22 times on this
        // part (cudaOccupancyMaxActiveClusters; 33 times for four, 45 for three), and with fewer, longer K loops the
        // two-kernel path below (CTA pairs on 256 x 256 tiles, partial sums through L2) was measured faster.
        const int units = (int)(ceil_div(m, kBM) * ceil_div(n, 192));
        if (units * 2 <= sms && units * 4 >= sms && g.kt_total >= 8) g.ck = 2;
    }
    if (g.ck) {
        g.bn = 192;
        g.pair = false;
        g.deep = false;
        g.tiles_m = (int)ceil_div(m, kBM);
        g.tiles_n = (int)ceil_div(n, g.bn);
        g.splits = 1;                                   // nothing goes through a workspace
        g.kt_per_split = (int)ceil_div(g.kt_total, g.ck);
        return g;
    }
    if (g.kt_total >= 3 && g.kt_total <= 4 && n >= 192 && m >= 2048 && sms >= 2 &&
        ceil_div(ceil_div(m, kBM), 2) * ceil_div(n, 192) >= sms) {
        // short contraction, tall output: pairs of CTAs walk down columns of 256 x 192 tiles with the column's B block resident
        // (with one or two K tiles the single-CTA B-stationary kernel below measured 4-10 % faster; with fewer than two pair
        // tiles per CTA pair the set-up of a column costs more than the kernel saves: 12.3 against 10.2 us at 2048 x 768 x 768)
        g.pbs = true;
        g.bn = 192;
        g.pair = false;
        g.deep = false;
        g.tiles_m = (int)ceil_div(m, kBM);
        g.tiles_n = (int)ceil_div(n, g.bn);
        g.splits = 1;
        g.kt_per_split = g.kt_total;
        return g;
    }
    if (g.kt_total <= 2 && n > 128) {
        // the whole B block of a tile column fits in shared memory next to a deep ring of A tiles.  (Instances for up to
        // four and six K tiles, whose rings hold barely more than one tile, measured no faster than the kernel above.)
        g.bs = 1;
        g.bn = 192;
        g.pair = false;
        g.deep = false;
        g.tiles_m = (int)ceil_div(m, kBM);
        g.tiles_n = (int)ceil_div(n, g.bn);
        g.splits = 1;
        g.kt_per_split = g.kt_total;
        return g;
    }
    if (n <= 128) g.bn = 128;
    else if (kc <= 1024 || n < 256 || (kc <= 2304 && n % 256 != 0 && n % 192 == 0)) g.bn = 192;
    else g.bn = 256;
    g.pair = g.bn == 256 && m > 128 && sms >= 2;
    g.tiles_m = (int)ceil_div(m, kBM);
    g.tiles_n = (int)ceil_div(n, g.bn);
    const int units = (g.pair ? (g.tiles_m + 1) / 2 : g.tiles_m) * g.tiles_n;   // work items before splitting K
    const int workers = g.pair ? sms / 2 : sms;
    int splits = 1;
    if (allow_split && units * 2 <= workers && g.kt_total >= 8) {
        splits = min(workers / units, g.kt_total / 4);
        splits = max(1, min(splits, 32));
    }
    g.kt_per_split = (int)ceil_div(g.kt_total, splits);
    g.splits = (int)ceil_div(g.kt_total, g.kt_per_split);
    g.deep = g.kt_per_split <= 8;   // K loop of at most 2048 per tile
    return g;
}

static bool ensure_device_ok()
{
    static int ok[kMaxDevices];   // 0 unknown, 1 yes, -1 no
    const int dev = current_device();
    if (dev < 0) return false;
    std::lock_guard<std::mutex> hold(g_dev_lock);
    if (!ok[dev]) {
        int major = 0;
        ok[dev] = (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess && major == 10) ? 1 : -1;
    }
    return ok[dev] == 1;
}

template <bool DEEP>
static mxfp4_status_t launch_gemm_pair(const CUtensorMap &ma, const CUtensorMap &mb, const CUtensorMap &msa, const CUtensorMap &msb,
                                       const CUtensorMap &md, const GemmParams &p, int grid, cudaStream_t st)
{
    using C = Gemm2Cfg<DEEP>;
    static bool attr_set[kMaxDevices];
    MX_CHECK_CUDA(set_smem_once(attr_set, k_gemm_mxf4_pair<DEEP>, C::kSmemBytes));
    k_gemm_mxf4_pair<DEEP><<<grid, kGemmThreads, C::kSmemBytes, st>>>(ma, mb, msa, msb, md, p);
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

template <int KT, int AS>
static mxfp4_status_t launch_gemm_pbs(const CUtensorMap &ma, const CUtensorMap &mb, const CUtensorMap &msa, const CUtensorMap &msb,
                                      const CUtensorMap &md, const CUtensorMap &mdw, const GemmParams &p, int grid, cudaStream_t st)
{
    using C = GemmPbsCfg<KT, AS>;
    if (p.kt_total > KT) return MXFP4_INVALID_ARG;   // the resident block holds KT K tiles
    static bool attr_set[kMaxDevices];
    MX_CHECK_CUDA(set_smem_once(attr_set, k_gemm_mxf4_pbs<KT, AS>, C::kSmemBytes));
    k_gemm_mxf4_pbs<KT, AS><<<grid, kGemmThreads, C::kSmemBytes, st>>>(ma, mb, msa, msb, md, mdw, p);
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

template <int BN, int KT, int AS>
static mxfp4_status_t launch_gemm_bs(const CUtensorMap &ma, const CUtensorMap &mb, const CUtensorMap &md, const CUtensorMap &mdw,
                                     const GemmParams &p, int grid, cudaStream_t st)
{
    using C = GemmBsCfg<BN, KT, AS>;
    static bool attr_set[kMaxDevices];
    MX_CHECK_CUDA(set_smem_once(attr_set, k_gemm_mxf4_bs<BN, KT, AS>, C::kSmemBytes));
    k_gemm_mxf4_bs<BN, KT, AS><<<grid, kGemmThreads, C::kSmemBytes, st>>>(ma, mb, md, mdw, p);
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

static mxfp4_status_t launch_gemm_ck(const CUtensorMap &ma, const CUtensorMap &mb, const GemmParams &p, int tiles, int cluster,
                                     cudaStream_t st)
{
    using C = GemmCkCfg;
    static bool attr_set[kMaxDevices];
    MX_CHECK_CUDA(set_smem_once(attr_set, k_gemm_mxf4_ck, C::kSmemBytes));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(tiles * cluster));
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    MX_CHECK_CUDA(cudaLaunchKernelEx(&cfg, k_gemm_mxf4_ck, ma, mb, p));
    MX_LAUNCHED();
    return MXFP4_OK;
}

template <int BN, bool DEEP>
static mxfp4_status_t launch_gemm(const CUtensorMap &ma, const CUtensorMap &mb, const CUtensorMap &md, const CUtensorMap &mdw,
                                  const GemmParams &p, int grid, cudaStream_t st)
{
    using C = GemmCfg<BN, DEEP>;
    static bool attr_set[kMaxDevices];
    MX_CHECK_CUDA(set_smem_once(attr_set, k_gemm_mxf4<BN, DEEP>, C::kSmemBytes));
    k_gemm_mxf4<BN, DEEP><<<grid, kGemmThreads, C::kSmemBytes, st>>>(ma, mb, md, mdw, p);
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

// Everything gemm() checks before it enqueues anything, without enqueuing anything: callers that launch other kernels
// first (the linear layer) ask here so that an error leaves the stream untouched.  allow_split = false: plan without
// split-K (no workspace needed).
mxfp4_status_t gemm_check(mxfp4_mat_t a, mxfp4_mat_t b, const void *d, int64_t ldd, int out_dtype, const void *bias,
                          const void *workspace, size_t workspace_bytes, bool allow_split)
{
    if (!a.data || !a.scales || !b.data || !b.scales || !d) return MXFP4_INVALID_ARG;
    if (out_dtype != MXFP4_OUT_BF16 && out_dtype != MXFP4_OUT_FP32) return MXFP4_INVALID_ARG;
    if (a.rows < 0 || b.rows < 0 || a.cols < 0) return MXFP4_INVALID_ARG;
    if (a.cols != b.cols || a.cols % 32 != 0 || b.rows % 8 != 0 || ldd < b.rows) return MXFP4_BAD_SHAPE;
    const int esz = out_dtype == MXFP4_OUT_FP32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(a.data) | reinterpret_cast<uintptr_t>(b.data) | reinterpret_cast<uintptr_t>(a.scales) |
         reinterpret_cast<uintptr_t>(b.scales) | reinterpret_cast<uintptr_t>(d) | reinterpret_cast<uintptr_t>(bias)) & 15u)
        return MXFP4_MISALIGNED;
    if ((ldd * esz) % 16 != 0) return MXFP4_MISALIGNED;
    const int64_t M = a.rows, N = b.rows, Kc = a.cols;
    if (M == 0 || N == 0) return MXFP4_OK;
    if (!ensure_device_ok()) return MXFP4_UNSUPPORTED_DEVICE;
    if (Kc == 0) return MXFP4_BAD_SHAPE;
    const GemmPlan g = plan_gemm(M, N, Kc, sm_count(), allow_split);
    const size_t need = g.splits > 1 ? (size_t)g.splits * M * N * sizeof(float) : 0;
    if (need > 0 && (!workspace || workspace_bytes < need)) return MXFP4_WORKSPACE_TOO_SMALL;
    if (need > 0 && (reinterpret_cast<uintptr_t>(workspace) & 15u)) return MXFP4_MISALIGNED;
    return MXFP4_OK;
}

// spin_limit / withhold_loads: see GemmParams (normal use: kWaitSpinLimit, 0).
static mxfp4_status_t gemm_impl(mxfp4_mat_t a, mxfp4_mat_t b, void *d, int64_t ldd, int out_dtype, const void *bias, void *workspace,
                                size_t workspace_bytes, uint32_t *dev_status, cudaStream_t st, bool allow_split, uint32_t spin_limit,
                                int withhold_loads)
{
    const mxfp4_status_t chk = gemm_check(a, b, d, ldd, out_dtype, bias, workspace, workspace_bytes, allow_split);
    if (chk) return chk;
    const int64_t M = a.rows, N = b.rows, Kc = a.cols;
    if (M == 0 || N == 0) return MXFP4_OK;
    const int sms = sm_count();
    const GemmPlan g = plan_gemm(M, N, Kc, sms, allow_split);

    const bool store_fp32 = g.splits > 1 || out_dtype == MXFP4_OUT_FP32;
    CUtensorMap ma, mb, md;
    if (!make_operand_map(&ma, a.data, M, Kc, kBM) || !make_operand_map(&mb, b.data, N, Kc, g.pbs ? 96 : g.pair ? 128 : g.bn)) return MXFP4_CUDA_ERROR;
    if (!make_output_map(&md, g.splits > 1 ? workspace : d, M, N, g.splits > 1 ? N : ldd, g.splits, store_fp32)) return MXFP4_CUDA_ERROR;

    GemmParams p;
    p.sfa = a.scales; p.sfb = b.scales;
    p.M = M; p.N = N; p.Kc = Kc;
    p.nblk4 = (int)ceil_div(Kc / 32, 4);
    p.rbA = (int)ceil_div(M, 128); p.rbB = (int)ceil_div(N, 128);
    p.tiles_m = g.tiles_m; p.tiles_n = g.tiles_n; p.splits = g.splits;
    p.kt_total = g.kt_total; p.kt_per_split = g.kt_per_split;
    p.out_fp32 = store_fp32;
    p.bias = static_cast<const __nv_bfloat16 *>(bias);
    p.dev_status = dev_status;
    p.d = d;
    p.ldd = ldd;
    p.spin_limit = spin_limit;
    p.withhold_loads = withhold_loads;
    if (g.ck) {
        p.splits = g.ck;
        p.out_fp32 = out_dtype == MXFP4_OUT_FP32;
        return launch_gemm_ck(ma, mb, p, g.tiles_m * g.tiles_n, g.ck, st);
    }
    const bool paired = g.pair || g.pbs;
    const int items = (paired ? (g.tiles_m + 1) / 2 : g.tiles_m) * g.tiles_n * g.splits;
    const int grid = paired ? 2 * min(items, sms / 2) : min(items, sms);
    CUtensorMap msa, msb;
    if (paired && (!make_scale_map(&msa, a.scales, M, Kc, 1) || !make_scale_map(&msb, b.scales, N, Kc, 2))) return MXFP4_CUDA_ERROR;
    CUtensorMap mdw = md;
    if (!store_fp32 && !make_output_map_wide(&mdw, d, M, N, ldd)) return MXFP4_CUDA_ERROR;
    mxfp4_status_t s = g.pbs         ? launch_gemm_pbs<4, 8>(ma, mb, msa, msb, md, mdw, p, grid, st)
                       : g.bs == 1   ? launch_gemm_bs<192, 2, 7>(ma, mb, md, mdw, p, grid, st)
                       : g.pair      ? (g.deep ? launch_gemm_pair<true>(ma, mb, msa, msb, md, p, grid, st) : launch_gemm_pair<false>(ma, mb, msa, msb, md, p, grid, st))
                       : g.bn == 256 ? (g.deep ? launch_gemm<256, true>(ma, mb, md, mdw, p, grid, st) : launch_gemm<256, false>(ma, mb, md, mdw, p, grid, st))
                       : g.bn == 192 ? launch_gemm<192, false>(ma, mb, md, mdw, p, grid, st)
                                     : (g.deep ? launch_gemm<128, true>(ma, mb, md, mdw, p, grid, st) : launch_gemm<128, false>(ma, mb, md, mdw, p, grid, st));
    if (s) return s;
    if (g.splits > 1 && !withhold_loads) {
        const int64_t total4 = M * N / 4;
        const int64_t nb4 = ceil_div(total4, 256);
        const int blocks = (int)(nb4 < (int64_t)sms * 8 ? nb4 : (int64_t)sms * 8);
        k_splitk_reduce<<<blocks, 256, 0, st>>>(static_cast<const float *>(workspace), g.splits, M, N, d, ldd,
                                                out_dtype == MXFP4_OUT_FP32, static_cast<const __nv_bfloat16 *>(bias));
        MX_CHECK_LAUNCH();
    }
    return MXFP4_OK;
}

mxfp4_status_t gemm(mxfp4_mat_t a, mxfp4_mat_t b, void *d, int64_t ldd, int out_dtype, const void *bias, void *workspace,
                    size_t workspace_bytes, uint32_t *dev_status, cudaStream_t st, bool allow_split)
{
    return gemm_impl(a, b, d, ldd, out_dtype, bias, workspace, workspace_bytes, dev_status, st, allow_split, kWaitSpinLimit, 0);
}

// bf16 matrix [m, n] (leading dimension ld) as a 2-D tensor; box = 64 columns x 128 rows, 128B swizzle: one half of the
// quantizing kernel's tile.
static bool make_tile_map_bf16(CUtensorMap *map, void *d, int64_t m, int64_t n, int64_t ld)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)n, (cuuint64_t)m};
    cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    cuuint32_t estr[2] = {1, 1};
    return encode_tiled_cached(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, d, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// packed transposed codes [n, m / 2 bytes]; box = 64 bytes x 128 rows, 64B swizzle (the column pass's staging tile)
static bool make_codes_t_map(CUtensorMap *map, void *packed, int64_t m, int64_t n)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)(m / 2), (cuuint64_t)n};
    cuuint64_t gstride[1] = {(cuuint64_t)(m / 2)};
    cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    cuuint32_t estr[2] = {1, 1};
    return encode_tiled_cached(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, packed, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
              CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static QuantSide make_quant_side(const mxfp4_mat_t &m, const mxfp4_qparams_t &qp)
{
    QuantSide s;
    s.packed = static_cast<uint8_t *>(m.data);
    s.scales = m.scales;
    s.nblk4 = (int)ceil_div(m.cols / 32, 4);
    s.scale_mode = qp.scale_mode;
    s.sr = make_sr_stream(qp.seed, qp.stream_id);
    return s;
}

template <bool SR_ROW, bool SR_T, bool DQ, bool WITH_Y>
static mxfp4_status_t launch_gemm_q(const CUtensorMap &ma, const CUtensorMap &mb, const CUtensorMap &my, const CUtensorMap &mz,
                                    const CUtensorMap &mx_, const CUtensorMap &mt, const GemmParams &p, const QuantEpilogue &e, int grid,
                                    cudaStream_t st)
{
    using C = GemmQCfg<WITH_Y>;
    static bool attr_set[kMaxDevices];
    MX_CHECK_CUDA(set_smem_once(attr_set, k_gemm_mxf4_q<SR_ROW, SR_T, DQ, WITH_Y>, C::kSmemBytes));
    k_gemm_mxf4_q<SR_ROW, SR_T, DQ, WITH_Y><<<grid, kGemmThreads, C::kSmemBytes, st>>>(ma, mb, my, mz, mx_, mt, p, e);
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

static bool valid_qp(const mxfp4_qparams_t &qp)
{
    return (qp.scale_mode == MXFP4_SCALE_TRUNCATION_FREE || qp.scale_mode == MXFP4_SCALE_FLOOR) &&
           (qp.rounding == MXFP4_ROUND_NEAREST || qp.rounding == MXFP4_ROUND_STOCHASTIC);
}

// Everything gemm_quant() checks, without enqueuing anything.
mxfp4_status_t gemm_quant_check(mxfp4_mat_t a, mxfp4_mat_t b, const void *bias, const mxfp4_epilogue_t *epi)
{
    if (!epi || !a.data || !a.scales || !b.data || !b.scales) return MXFP4_INVALID_ARG;
    if (a.rows < 0 || b.rows < 0 || a.cols < 0) return MXFP4_INVALID_ARG;
    if (epi->hook != MXFP4_HOOK_IDENTITY && epi->hook != MXFP4_HOOK_GELU && epi->hook != MXFP4_HOOK_MULTIPLY) return MXFP4_INVALID_ARG;
    const int64_t M = a.rows, N = b.rows, Kc = a.cols;
    const bool row = epi->zq.data != nullptr, tr = epi->zq_t.data != nullptr;
    if (!row && !tr && !epi->y_bf16 && !epi->z_bf16) return MXFP4_INVALID_ARG;
    if (epi->chain && !(row && tr)) return MXFP4_INVALID_ARG;
    if (epi->hook == MXFP4_HOOK_MULTIPLY && !epi->aux_bf16) return MXFP4_INVALID_ARG;
    if ((row && (!epi->zq.scales || !valid_qp(epi->qp_row))) || (tr && (!epi->zq_t.scales || !valid_qp(epi->qp_t)))) return MXFP4_INVALID_ARG;
    if (a.cols != b.cols || Kc % 32 != 0 || N % 32 != 0 || (tr && M % 32 != 0)) return MXFP4_BAD_SHAPE;
    if (M > 0x7FFFFF80 || N > 0x7FFFFF80) return MXFP4_BAD_SHAPE;
    if (row && (epi->zq.rows != M || epi->zq.cols != N)) return MXFP4_BAD_SHAPE;
    if (tr && (epi->zq_t.rows != N || epi->zq_t.cols != M)) return MXFP4_BAD_SHAPE;
    if ((epi->y_bf16 && epi->ldy < N) || (epi->z_bf16 && epi->ldz < N) || (epi->hook == MXFP4_HOOK_MULTIPLY && epi->ld_aux < N)) return MXFP4_BAD_SHAPE;
    uintptr_t bits = reinterpret_cast<uintptr_t>(a.data) | reinterpret_cast<uintptr_t>(b.data) | reinterpret_cast<uintptr_t>(a.scales) |
                     reinterpret_cast<uintptr_t>(b.scales) | reinterpret_cast<uintptr_t>(bias) | reinterpret_cast<uintptr_t>(epi->y_bf16) |
                     reinterpret_cast<uintptr_t>(epi->z_bf16);
    if (epi->hook == MXFP4_HOOK_MULTIPLY) bits |= reinterpret_cast<uintptr_t>(epi->aux_bf16);
    if (row) bits |= reinterpret_cast<uintptr_t>(epi->zq.data) | reinterpret_cast<uintptr_t>(epi->zq.scales);
    if (tr) bits |= reinterpret_cast<uintptr_t>(epi->zq_t.data) | reinterpret_cast<uintptr_t>(epi->zq_t.scales);
    if (bits & 15u) return MXFP4_MISALIGNED;
    if ((epi->y_bf16 && epi->ldy % 8) || (epi->z_bf16 && epi->ldz % 8) || (epi->hook == MXFP4_HOOK_MULTIPLY && epi->ld_aux % 8)) return MXFP4_MISALIGNED;
    if (M == 0 || N == 0) return MXFP4_OK;
    if (!ensure_device_ok()) return MXFP4_UNSUPPORTED_DEVICE;
    if (Kc == 0) return MXFP4_BAD_SHAPE;
    return MXFP4_OK;
}

mxfp4_status_t gemm_quant(mxfp4_mat_t a, mxfp4_mat_t b, const void *bias, const mxfp4_epilogue_t *epi, uint32_t *dev_status, cudaStream_t st)
{
    const mxfp4_status_t chk = gemm_quant_check(a, b, bias, epi);
    if (chk) return chk;
    const int64_t M = a.rows, N = b.rows, Kc = a.cols;
    if (M == 0 || N == 0) return MXFP4_OK;
    const bool row = epi->zq.data != nullptr, tr = epi->zq_t.data != nullptr;
    CUtensorMap ma, mb, my, mz, mx_, mt;
    if (!make_operand_map(&ma, a.data, M, Kc, kBM) || !make_operand_map(&mb, b.data, N, Kc, 128)) return MXFP4_CUDA_ERROR;
    my = mz = mx_ = mt = ma;   // placeholders when the tensors they describe are not asked for
    if (epi->z_bf16 && !make_tile_map_bf16(&mz, epi->z_bf16, M, N, epi->ldz)) return MXFP4_CUDA_ERROR;
    if (tr && !make_codes_t_map(&mt, epi->zq_t.data, M, N)) return MXFP4_CUDA_ERROR;

    GemmParams p;
    p.sfa = a.scales; p.sfb = b.scales;
    p.M = M; p.N = N; p.Kc = Kc;
    p.nblk4 = (int)ceil_div(Kc / 32, 4);
    p.rbA = (int)ceil_div(M, 128); p.rbB = (int)ceil_div(N, 128);
    p.tiles_m = (int)ceil_div(M, kBM); p.tiles_n = (int)ceil_div(N, 128); p.splits = 1;
    p.kt_total = (int)ceil_div(Kc, kBKElems); p.kt_per_split = p.kt_total;
    p.out_fp32 = 0;
    p.bias = static_cast<const __nv_bfloat16 *>(bias);
    p.dev_status = dev_status;
    p.d = nullptr;
    p.ldd = 0;
    p.spin_limit = kWaitSpinLimit;
    p.withhold_loads = 0;

    QuantEpilogue e;
    const mxfp4_qparams_t none = {MXFP4_SCALE_TRUNCATION_FREE, MXFP4_ROUND_NEAREST, 0, 0, 0};
    const mxfp4_mat_t nomat = {nullptr, nullptr, 0, 32};
    e.rw = make_quant_side(row ? epi->zq : nomat, row ? epi->qp_row : none);
    e.tr = make_quant_side(tr ? epi->zq_t : nomat, tr ? epi->qp_t : none);
    e.emit_row = row; e.emit_t = tr;
    e.hook = epi->hook;
    e.aux = static_cast<const __nv_bfloat16 *>(epi->aux_bf16); e.ld_aux = epi->ld_aux;
    e.store_y = epi->y_bf16 != nullptr;
    e.store_z = epi->z_bf16 != nullptr;
    if (e.store_y && !make_tile_map_bf16(&my, epi->y_bf16, M, N, epi->ldy)) return MXFP4_CUDA_ERROR;
    if (e.hook == MXFP4_HOOK_IDENTITY && e.store_y && !e.store_z) {
        mz = my;         // Y = Z: one tile, one pair of stores
        e.store_y = 0;
        e.store_z = 1;
    }
    e.aux_tma = 0;
    if (e.hook == MXFP4_HOOK_MULTIPLY) {
        if (!make_tile_map_bf16(&mx_, const_cast<void *>(epi->aux_bf16), M, N, epi->ld_aux)) return MXFP4_CUDA_ERROR;
        e.aux_tma = 1;
    }
    const int items = p.tiles_m * p.tiles_n;
    const int sms = sm_count();
    const int grid = items < sms ? items : sms;
    const bool sr_r = row && epi->qp_row.rounding == MXFP4_ROUND_STOCHASTIC, sr_t = tr && epi->qp_t.rounding == MXFP4_ROUND_STOCHASTIC;
    const int sel = (e.store_y ? 8 : 0) | (epi->chain ? 4 : 0) | (sr_r ? 2 : 0) | (sr_t ? 1 : 0);
#define MX_Q_CASE(i, a_, b_, c_, d_) case i: return launch_gemm_q<a_, b_, c_, d_>(ma, mb, my, mz, mx_, mt, p, e, grid, st)
    switch (sel) {
    MX_Q_CASE(0, false, false, false, false);
    MX_Q_CASE(1, false, true, false, false);
    MX_Q_CASE(2, true, false, false, false);
    MX_Q_CASE(3, true, true, false, false);
    MX_Q_CASE(4, false, false, true, false);
    MX_Q_CASE(5, false, true, true, false);
    MX_Q_CASE(6, true, false, true, false);
    MX_Q_CASE(7, true, true, true, false);
    MX_Q_CASE(8, false, false, false, true);
    MX_Q_CASE(9, false, true, false, true);
    MX_Q_CASE(10, true, false, false, true);
    MX_Q_CASE(11, true, true, false, true);
    MX_Q_CASE(12, false, false, true, true);
    MX_Q_CASE(13, false, true, true, true);
    MX_Q_CASE(14, true, false, true, true);
    default: return launch_gemm_q<true, true, true, true>(ma, mb, my, mz, mx_, mt, p, e, grid, st);
    }
#undef MX_Q_CASE
}

size_t gemm_workspace_bytes(int64_t m, int64_t n, int64_t kc)
{
    if (m <= 0 || n <= 0 || kc <= 0) return 0;
    // the same SM count gemm() plans with (148, the B200's, when no device is current)
    const GemmPlan g = plan_gemm(m, n, kc, sm_count());
    return g.splits > 1 ? (size_t)g.splits * m * n * sizeof(float) : 0;
}

// The longest chain of MMAs (64 contraction elements each) that gemm() adds into one accumulator for this shape.
int64_t gemm_chain_mmas(int64_t m, int64_t n, int64_t kc)
{
    if (m <= 0 || n <= 0 || kc <= 0) return 0;
    const GemmPlan g = plan_gemm(m, n, kc, sm_count());
    const int64_t kt = g.ck ? (g.kt_per_split + 1) / 2 : g.kt_per_split;   // the cluster kernel alternates between two accumulators
    const int64_t elems = kt * kBKElems < kc ? kt * kBKElems : kc;
    return ceil_div(elems, 64);
}

}  // namespace mx

extern "C" {

int64_t mxfp4_gemm_chain_mmas(int64_t m, int64_t n, int64_t kc) { return mx::gemm_chain_mmas(m, n, kc); }

mxfp4_status_t mxfp4_mma_issue_ceiling(int32_t bn, int32_t iters, uint32_t *dev_status, void *stream)
{
    if (iters < 1 || iters > (1 << 24) || (bn != 128 && bn != 192 && bn != 256)) return MXFP4_INVALID_ARG;
    if (!mx::ensure_device_ok()) return MXFP4_UNSUPPORTED_DEVICE;
    const int smem = mx::kBM * mx::kBKBytes + bn * mx::kBKBytes + 2 * mx::kSfChunk * (1 + (bn + 127) / 128) + 1024 + 256;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int grid = mx::sm_count();
    if (bn == 128) {
        MX_CHECK_CUDA(cudaFuncSetAttribute(mx::k_mma_ceiling<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        mx::k_mma_ceiling<128><<<grid, 128, smem, st>>>(iters, dev_status);
    } else if (bn == 192) {
        MX_CHECK_CUDA(cudaFuncSetAttribute(mx::k_mma_ceiling<192>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        mx::k_mma_ceiling<192><<<grid, 128, smem, st>>>(iters, dev_status);
    } else {
        MX_CHECK_CUDA(cudaFuncSetAttribute(mx::k_mma_ceiling<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        mx::k_mma_ceiling<256><<<grid, 128, smem, st>>>(iters, dev_status);
    }
    MX_CHECK_LAUNCH();
    return MXFP4_OK;
}

size_t mxfp4_gemm_workspace_bytes(int64_t m, int64_t n, int64_t kc) { return mx::gemm_workspace_bytes(m, n, kc); }

mxfp4_status_t mxfp4_gemm_quant(mxfp4_mat_t a, mxfp4_mat_t b, const void *bias_bf16, const mxfp4_epilogue_t *epi, uint32_t *dev_status,
                                void *stream)
{
    return mx::gemm_quant(a, b, bias_bf16, epi, dev_status, static_cast<cudaStream_t>(stream));
}

mxfp4_status_t mxfp4_gemm_wait_selftest(mxfp4_mat_t a, mxfp4_mat_t b, void *d, int64_t ldd, int32_t out_dtype, void *workspace,
                                        size_t workspace_bytes, uint32_t spin_limit, uint32_t *dev_status, void *stream)
{
    if (!dev_status || spin_limit < 128u || spin_limit > (1u << 16)) return MXFP4_INVALID_ARG;
    return mx::gemm_impl(a, b, d, ldd, out_dtype, nullptr, workspace, workspace_bytes, dev_status, static_cast<cudaStream_t>(stream), true,
                         spin_limit, 1);
}

mxfp4_status_t mxfp4_gemm(mxfp4_mat_t a, mxfp4_mat_t b, void *d, int64_t ldd, int32_t out_dtype, const void *bias_bf16,
                          void *workspace, size_t workspace_bytes, uint32_t *dev_status, void *stream)
{
    return mx::gemm(a, b, d, ldd, out_dtype, bias_bf16, workspace, workspace_bytes, dev_status, static_cast<cudaStream_t>(stream), true);
}

}  // extern "C"
