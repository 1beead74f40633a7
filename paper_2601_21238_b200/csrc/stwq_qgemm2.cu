// qgemm2: the main int8 GEMM + dequantize epilogue, as CTA pairs (tcgen05 cta_group::2).
//
//   acc[m,n] = sum_k Xq[m,k] * Wq[n,k]                              (Section 3, Y = X W on codes)
//   Y[m,n]   = act( float(acc) * (s_tok[pos[m]] * s_w[n]) + bias[n] )   (Appendix A.1 dequantizer)
//
// A cluster of two CTAs (two SMs) owns a 256 x BN output tile. Each CTA loads its own 128 rows
// of Xq and its own half (BN/2 rows) of the Wq slice with TMA; one thread of the even CTA issues
// tcgen05.mma.cta_group::2 (M = 256, N = BN, K = 32), which reads both CTAs' shared memory, so
// every byte of Wq is staged once per pair instead of once per SM. Each CTA's tensor memory holds
// the accumulator rows of its own 128 rows, in two buffers of BN columns so that the next tile's
// main loop runs while this tile drains.
//
// Roles per CTA (kThreads = 64 + 32 * EPI threads):
//   warp 0          TMA producer (one lane): ring of STAGES stages; completion bytes of both CTAs
//                   land on the even CTA's "full" barrier
//   warp 1          MMA issuer (one lane, even CTA only); tcgen05.commit multicasts "stage free"
//                   and "accumulator full" to both CTAs
//   warps 2..2+EPI  epilogue: tcgen05.ld (the next chunk's loads in flight while this one is
//                   converted; the accumulator is handed back as soon as the last load has
//                   landed) -> packed fp32 scale/bias/GELU -> convert -> either a 128-byte-swizzled
//                   staging tile in shared memory and a TMA store (full-line writes, clipped at
//                   the matrix edge by the tensor map) or 256-bit stores straight from registers.
//                   Warp w may read TMEM lanes 32*(w%4)..+31; with EPI = 8 two warps share a lane
//                   quarter and alternate column chunks.
// Every mbarrier wait is bounded (limit in ns from the host); on expiry the CTA raises
// STWQ_DEV_TIMEOUT, all roles leave their loops, loads in flight are awaited with the same
// bound, both CTAs meet at the cluster barrier, tensor memory is freed and the kernel returns.
#include "stwq_internal.cuh"
#include "stwq_ptx.cuh"

using namespace stwq_ptx;

namespace {

constexpr int kBM = 128;      // rows per CTA
constexpr int kBK = 128;      // bytes of K per stage
constexpr int kOutCodes = 3;  // internal output type: int8 codes for the next layer (see stwq_chain)

struct Gemm2Params {
    int64_t M;
    int N, K, P;
    const int32_t* pos_ids;
    const float* s_w;
    const float* s_tok;
    const float* bias;
    int tiles_n, num_tiles, num_kb;
    uint32_t* status;
    unsigned long long wait_limit_ns;
    // Work units: the first `full_units` are whole tiles; then the last `tail_tiles` tiles come
    // as `nsplit` units each, one per range of kb_per_split k-blocks (split-K for the last,
    // partly filled wave). num_units = full_units + tail_tiles * nsplit.
    int full_units, num_units, nsplit, kb_per_split;
    int32_t* partial;          // [tail tile][split][rank][warp][128 x 32 lanes] int32
    uint32_t* counters;        // [tail tile][rank][warp]
    // asymmetric quantizer (ASYM): acc - z_w[n] rowcorr[m] - z_tok[pos] colsum[n] replaces acc
    const int32_t* z_tok;      // [P]
    const int32_t* z_w;        // [N]
    const int32_t* colsum;     // [N]
    const int32_t* rowcorr;    // [M]
    // chained output (OUT == kOutCodes): the next layer's static quantizer applied to act(z)
    const float* s_ch_next;    // [N] or NULL
    const float* s_tok_next;   // [P]
    int qmin_next, qmax_next;
    void* Y;                   // used by the direct-store epilogue
    int y_vec32;               // Y base and row pitch are 32-byte aligned: 256-bit stores are legal
    // batched operands (attention heads): tile index = g * tiles_per_g + tile within matrix g
    int tiles_per_g;
    int pos_shared;            // pos_ids indexed by the row within the matrix (else by g * M + row)
    int64_t sw_gstride;        // s_w of matrix g starts at s_w + g * sw_gstride
    uint32_t idesc;            // instruction descriptor (signed or unsigned A)
};

// STORE = 0: the epilogue stages 32 x 128-byte pieces in shared memory and writes them with TMA
// (the fewest shared-memory cycles per output byte; best when K is small and the epilogue is
// as long as the main loop). STORE = 1: every thread writes its row's 128 bytes straight from
// registers with 256-bit stores; no staging memory, so the operand ring can be deeper.
template <int BN, int STAGES, int EPI, int STORE>
struct Smem2 {
    static constexpr int kABytes = kBM * kBK;               // 16 KB
    static constexpr int kBBytes = (BN / 2) * kBK;          // this CTA's half of the Wq slice
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kOffB = STAGES * kABytes;
    static constexpr int kOffStage = STAGES * kStageBytes;  // per epilogue warp: two staging tiles of 32 rows x 128 B
    static constexpr int kOffScale = kOffStage + (STORE == 0 ? EPI * 8192 : 0); // per epilogue warp: s_w and bias of its columns
    static constexpr int kOffBars = kOffScale + 4 * BN * 4 * 4;   // s_w, bias, and either the next layer's 1 / s_ch (chained
                                                                  // output) or the weights' zero points and code sums (asymmetric)
    static constexpr int kNumBars = 2 * STAGES + 4;
    static constexpr int kOffMisc = kOffBars + kNumBars * 8;
    static constexpr int kTotal = kOffMisc + 16;
    static constexpr int kDynamic = kTotal + 1024;
    static_assert(kDynamic <= 227 * 1024, "shared memory budget");
};

// ---------------------------------------------------------------------------- kernel
// OUT: element type of Y (STWQ_OUT_*); ACT: activation. One staging chunk is 32 rows x 128 bytes:
// 64 bf16 columns or 32 fp32 / int32 columns.
struct Unit {
    int tile, kb0, kb1, split, tail;    // tail = index among the split tiles, -1 for a whole tile
};
__device__ __forceinline__ Unit decode_unit(const Gemm2Params& p, int u)
{
    Unit w;
    if (u < p.full_units) {
        w.tile = u; w.kb0 = 0; w.kb1 = p.num_kb; w.split = 0; w.tail = -1;
    } else {
        const int j = u - p.full_units;
        w.tail = j / p.nsplit;
        w.split = j % p.nsplit;
        w.tile = p.full_units + w.tail;
        w.kb0 = w.split * p.kb_per_split;
        w.kb1 = min(w.kb0 + p.kb_per_split, p.num_kb);
    }
    return w;
}
__device__ __forceinline__ uint4 ld_cg_v4(const void* ptr)
{
    uint4 v;
    asm volatile("ld.global.cg.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(ptr) : "memory");
    return v;
}

// STORE: see Smem2. ASYM: zero-point correction of the accumulators (Eq. 1 with zero points).
template <int BN, int STAGES, int EPI, int OUT, int ACT, int STORE, bool ASYM>
__global__ void __launch_bounds__(64 + 32 * EPI, 1)
qgemm2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
              const __grid_constant__ CUtensorMap tmY, const Gemm2Params p)
{
    using L = Smem2<BN, STAGES, EPI, STORE>;
    constexpr int kChunkCols = (OUT == STWQ_OUT_BF16) ? 64 : (OUT == kOutCodes ? 128 : 32);
    constexpr int kChunks = BN / kChunkCols;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);

    const uint32_t bars = base + L::kOffBars;
    auto bar_full = [&](int s) { return bars + 8u * s; };
    auto bar_empty = [&](int s) { return bars + 8u * (STAGES + s); };
    auto bar_tfull = [&](int a) { return bars + 8u * (2 * STAGES + a); };
    auto bar_tempty = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kOffMisc);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::kOffMisc + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may queue up behind this grid
    const uint32_t rank = cluster_ctarank();            // 0 = even CTA = MMA leader
    const int pair = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full(s), 1);                   // leader's producer arrives with expect_tx
            mbar_init(bar_empty(s), 1);                  // multicast commit
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull(a), 1);                  // multicast commit
            mbar_init(bar_tempty(a), 2 * EPI);           // every epilogue warp of both CTAs
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(2 * BN)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                  // barriers of both CTAs are initialised
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const unsigned long long limit = p.wait_limit_ns;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // Two lanes issue the two loads of a stage in the same instruction: lane 0 the Xq rows,
        // lane 1 the Wq rows. One thread issuing both one after the other needs about 160 ns per
        // request (wait, expect, issue form a dependent chain), i.e. more than the 256 x 256 x 128
        // tile's 260 ns of tensor-pipe time per k-block; side by side the chain is paid once.
        if (lane < 2) {
            uint32_t it = 0;
            bool ok = true;
            const uint32_t full0 = mapa_u32(bar_full(0), 0);     // leader's barriers
            const CUtensorMap* my_map = lane == 0 ? &tmA : &tmB;
            const uint32_t my_dst0 = lane == 0 ? base : base + L::kOffB;
            const uint32_t my_stage_bytes = lane == 0 ? L::kABytes : L::kBBytes;
            // launched as a programmatic dependent of the quantize kernel: everything up to here
            // (barriers, tensor memory, cluster handshake) may have run while that kernel drained;
            // its codes are read only from here on
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int u = pair; ok && u < p.num_units; u += num_pairs) {
                const Unit w = decode_unit(p, u);
                const int g = w.tile / p.tiles_per_g;
                const int tile = w.tile - g * p.tiles_per_g;
                const int m0 = (tile / p.tiles_n) * (2 * kBM) + (int)rank * kBM;
                const int n0 = (tile % p.tiles_n) * BN + (int)rank * (BN / 2);
                const int my_row0 = lane == 0 ? m0 : n0;
                for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(bar_empty(s), ph ^ 1u, abort_flag, limit)) { ok = false; break; }
                    if (rank == 0 && lane == 0) mbar_expect_tx(bar_full(s), 2 * L::kStageBytes);
                    tma_load_3d_pair(my_dst0 + s * my_stage_bytes, my_map, kb * kBK, my_row0, g, full0 + 8u * s);
                }
            }
            ok = __all_sync(0x3u, ok);
            if (!ok && rank == 0 && lane == 0) {
                const uint32_t first = it > (uint32_t)STAGES ? it - STAGES : 0u;
                for (uint32_t j = first; j < it; ++j) {
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(bar_full(j % STAGES), (j / STAGES) & 1u))
                        if (globaltimer_ns() - t0 > limit) break;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader)
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = p.idesc;
            uint32_t it = 0, t = 0;
            bool ok = true;
            for (int u = pair; ok && u < p.num_units; u += num_pairs, ++t) {
                const Unit w = decode_unit(p, u);
                const int acc = t & 1;
                const uint32_t aph = (t >> 1) & 1u;
                if (!mbar_wait(bar_tempty(acc), aph ^ 1u, abort_flag, limit)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(bar_full(s), ph, abort_flag, limit)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = make_smem_desc(base + s * L::kABytes);
                    const uint64_t b_desc = make_smem_desc(base + L::kOffB + s * L::kBBytes);
#pragma unroll
                    for (int k = 0; k < kBK / 32; ++k)
                        tc_mma_i8_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb != w.kb0 || k != 0) ? 1u : 0u);
                    tc_commit_pair(bar_empty(s));
                }
                if (ok) tc_commit_pair(bar_tfull(acc));
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        // the asymmetric epilogue reads the row corrections that the quantize kernel accumulates
        if (ASYM) asm volatile("griddepcontrol.wait;" ::: "memory");
        const int ew = warp - 2;                          // 0..EPI-1
        const int q = warp & 3;                           // TMEM lane quarter
        const int sub = ew >> 2;                          // which of the EPI/4 warps of this quarter
        constexpr int kSubs = EPI / 4;
        constexpr int kMyChunks = kChunks / kSubs;        // column chunks this warp owns per tile
        constexpr int kMyCols = kMyChunks * kChunkCols;
        static_assert(kChunks % kSubs == 0, "chunks must divide among the warps of a quarter");
        const uint32_t stage0 = base + L::kOffStage + (uint32_t)ew * 8192u;   // two staging tiles (STORE == 0)
        float* my_sw = reinterpret_cast<float*>(smem + L::kOffScale) + ew * 4 * kMyCols;
        float* my_bias = my_sw + kMyCols;
        float* my_rcn = my_bias + kMyCols;
        int* my_zw = reinterpret_cast<int*>(my_rcn);       // asymmetric: the third and fourth arrays hold integers
        int* my_cs = my_zw + kMyCols;
        const uint32_t tempty0 = mapa_u32(bar_tempty(0), 0);
        constexpr int kElem = (OUT == STWQ_OUT_BF16) ? 2 : (OUT == kOutCodes ? 1 : 4);
        uint32_t t = 0, nstore = 0;
        bool ok = true;
        for (int u = pair; u < p.num_units; u += num_pairs, ++t) {
            const Unit wu = decode_unit(p, u);
            const int g = wu.tile / p.tiles_per_g;
            const int tile = wu.tile - g * p.tiles_per_g;
            const int acc = t & 1;
            const uint32_t aph = (t >> 1) & 1u;
            const int m0 = (tile / p.tiles_n) * (2 * kBM) + (int)rank * kBM;
            const int n0 = (tile % p.tiles_n) * BN;
            const int64_t row = (int64_t)m0 + q * 32 + lane;              // row within matrix g
            const int64_t grow = (int64_t)g * p.M + row;                  // row of the stacked output
            const int64_t prow = p.pos_shared ? row : grow;               // index into pos_ids
            const float* g_sw = p.s_w + (int64_t)g * p.sw_gstride;
            float st = 0.0f, rtn = 0.0f;
            int zx = 0, Rm = 0;
            if (ASYM) {
                __syncwarp();
                for (int i = lane * 4; i < kMyCols; i += 128) {
                    const int k = i / kChunkCols;
                    const int col = n0 + (sub + k * kSubs) * kChunkCols + (i % kChunkCols);
                    int4 zw = make_int4(0, 0, 0, 0), cs = make_int4(0, 0, 0, 0);
                    if (col < p.N) {
                        zw = __ldg(reinterpret_cast<const int4*>(p.z_w + col));
                        cs = __ldg(reinterpret_cast<const int4*>(p.colsum + col));
                    }
                    *reinterpret_cast<int4*>(my_zw + i) = zw;
                    *reinterpret_cast<int4*>(my_cs + i) = cs;
                }
                if (row < p.M) {
                    const int pos = p.pos_ids[prow];
                    Rm = p.rowcorr[grow];
                    if (pos >= 0 && pos < p.P) zx = p.z_tok[pos];
                }
                __syncwarp();
            }
            if (OUT != STWQ_OUT_INT32) {
                // column scales and biases of this warp's chunks -> its private shared copy, and
                // the row scale, all fetched before the accumulator is waited for
                __syncwarp();
                for (int i = lane * 4; i < kMyCols; i += 128) {
                    const int k = i / kChunkCols;
                    const int col = n0 + (sub + k * kSubs) * kChunkCols + (i % kChunkCols);
                    float4 sw = make_float4(0.f, 0.f, 0.f, 0.f), bi = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (col < p.N) {                      // N is a multiple of 4: the float4 is in range
                        sw = __ldg(reinterpret_cast<const float4*>(g_sw + col));
                        if (p.bias != nullptr) bi = __ldg(reinterpret_cast<const float4*>(p.bias + col));
                    }
                    *reinterpret_cast<float4*>(my_sw + i) = sw;
                    *reinterpret_cast<float4*>(my_bias + i) = bi;
                    if (OUT == kOutCodes) {
                        float4 rn = make_float4(1.f, 1.f, 1.f, 1.f);
                        if (col < p.N && p.s_ch_next != nullptr) {
                            const float4 sn = __ldg(reinterpret_cast<const float4*>(p.s_ch_next + col));
                            rn = make_float4(__fdiv_rn(1.0f, sn.x), __fdiv_rn(1.0f, sn.y), __fdiv_rn(1.0f, sn.z), __fdiv_rn(1.0f, sn.w));
                        }
                        *reinterpret_cast<float4*>(my_rcn + i) = rn;
                    }
                }
                if (row < p.M) {
                    const int pos = p.pos_ids != nullptr ? p.pos_ids[prow] : 0;      // no positions: one scale for all rows
                    if (pos >= 0 && pos < p.P) {
                        st = p.s_tok[pos];
                        if (OUT == kOutCodes) rtn = __fdiv_rn(1.0f, p.s_tok_next[pos]);
                    } else {
                        atomicOr(p.status, STWQ_DEV_POS_RANGE);
                    }
                }
                __syncwarp();
            }
            if (ok) ok = mbar_wait(bar_tfull(acc), aph, abort_flag, limit);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN);
            // All of this warp's accumulator columns are fetched at once (kLoads x 32 registers) and
            // the buffer is handed back as soon as they have landed; conversion and stores follow
            // from registers. tcgen05.ld queues behind the tensor-core instructions already issued,
            // so one exposed wait per tile is the best that can be had.
            constexpr int kLoadsPerChunk = (OUT == STWQ_OUT_BF16) ? 2 : (OUT == kOutCodes ? 4 : 1);
            constexpr int kLoads = kMyChunks * kLoadsPerChunk;
            uint32_t racc[kLoads][32];
#pragma unroll
            for (int k = 0; k < kMyChunks; ++k) {
                const int c = sub + k * kSubs;
#pragma unroll
                for (int h = 0; h < kLoadsPerChunk; ++h)
                    tmem_ld32(taddr + (uint32_t)(c * kChunkCols + h * 32), racc[k * kLoadsPerChunk + h]);
            }
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(tempty0 + 8u * acc);
            if (wu.tail >= 0) {
                // One of nsplit partial sums of a tail tile: publish this warp's piece (lane-interleaved,
                // 512 contiguous bytes per instruction), then count arrivals; the last warp to arrive for
                // this piece adds all pieces up and carries on with the epilogue, the others are done.
                // No CTA waits for another, and the sum of integers does not depend on the order.
                constexpr int kPieceInts = kLoads * 32 * 32;
                const size_t piece0 = (((size_t)wu.tail * p.nsplit) * 2 + rank) * EPI + ew;
                const size_t piece_stride = (size_t)2 * EPI;
                int32_t* mine = p.partial + (piece0 + (size_t)wu.split * piece_stride) * kPieceInts;
#pragma unroll
                for (int l = 0; l < kLoads; ++l)
#pragma unroll
                    for (int g = 0; g < 8; ++g) st_global_v4(mine + ((size_t)(l * 8 + g) * 32 + lane) * 4, racc[l] + g * 4);
                __threadfence();
                __syncwarp();
                uint32_t* counter = p.counters + ((size_t)wu.tail * 2 + rank) * EPI + ew;
                uint32_t old = 0;
                if (lane == 0) {
                    old = atomicAdd(counter, 1u);
                    if (old == (uint32_t)p.nsplit - 1u) *counter = 0u;    // all have arrived: ready for the next call
                }
                old = __shfl_sync(0xffffffffu, old, 0);
                if (old != (uint32_t)p.nsplit - 1u) continue;
                __threadfence();
                for (int s2 = 0; s2 < p.nsplit; ++s2) {
                    if (s2 == wu.split) continue;         // this warp's own piece is still in its registers
                    const int32_t* src = p.partial + (piece0 + (size_t)s2 * piece_stride) * kPieceInts;
#pragma unroll
                    for (int l = 0; l < kLoads; ++l)
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            const uint4 a = ld_cg_v4(src + ((size_t)(l * 8 + g) * 32 + lane) * 4);
                            racc[l][g * 4 + 0] += a.x; racc[l][g * 4 + 1] += a.y; racc[l][g * 4 + 2] += a.z; racc[l][g * 4 + 3] += a.w;
                        }
                }
            }
#pragma unroll
            for (int k = 0; k < kMyChunks; ++k, ++nstore) {
                const int c = sub + k * kSubs;
                const int col0 = n0 + c * kChunkCols;
                const float* csw = my_sw + k * kChunkCols;
                const float* cbi = my_bias + k * kChunkCols;
                const uint32_t* r0 = racc[k * kLoadsPerChunk];
                const uint32_t* r1 = racc[k * kLoadsPerChunk + kLoadsPerChunk - 1];
                uint32_t w[32];                           // this row's 128 bytes of output
                const uint64_t st2 = pack_f2(st, st);
                if (ASYM) {
                    // zero-point correction of this chunk, exact in int32:
                    // acc - z_w[n] rowcorr[m] - z_tok[pos] colsum[n]
#pragma unroll
                    for (int h = 0; h < kLoadsPerChunk; ++h) {
                        uint32_t* r = racc[k * kLoadsPerChunk + h];
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const int4 zw = *reinterpret_cast<const int4*>(my_zw + k * kChunkCols + h * 32 + j);
                            const int4 cs = *reinterpret_cast<const int4*>(my_cs + k * kChunkCols + h * 32 + j);
                            r[j + 0] = (uint32_t)((int)r[j + 0] - zw.x * Rm - zx * cs.x);
                            r[j + 1] = (uint32_t)((int)r[j + 1] - zw.y * Rm - zx * cs.y);
                            r[j + 2] = (uint32_t)((int)r[j + 2] - zw.z * Rm - zx * cs.z);
                            r[j + 3] = (uint32_t)((int)r[j + 3] - zw.w * Rm - zx * cs.w);
                        }
                    }
                }
                if (OUT == kOutCodes) {
                    // y = act(z) stays in fp32 registers and goes straight through the next layer's
                    // static quantizer: (y * rc_next[n]) * rt_next[pos], round to nearest even, clamp, pack
                    const float* crn = my_rcn + k * kChunkCols;
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const uint32_t* r = racc[k * kLoadsPerChunk + h];
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 sw = *reinterpret_cast<const float4*>(csw + h * 32 + j);
                            const float4 bi = *reinterpret_cast<const float4*>(cbi + h * 32 + j);
                            const float4 rn = *reinterpret_cast<const float4*>(crn + h * 32 + j);
                            uint64_t z01 = fma_f2(pack_f2((float)(int32_t)r[j + 0], (float)(int32_t)r[j + 1]),
                                                  mul_f2(st2, pack_f2(sw.x, sw.y)), pack_f2(bi.x, bi.y));
                            uint64_t z23 = fma_f2(pack_f2((float)(int32_t)r[j + 2], (float)(int32_t)r[j + 3]),
                                                  mul_f2(st2, pack_f2(sw.z, sw.w)), pack_f2(bi.z, bi.w));
                            z01 = apply_act_f2<ACT>(z01);
                            z23 = apply_act_f2<ACT>(z23);
                            float v0, v1, v2, v3;
                            unpack_f2(z01, v0, v1);
                            unpack_f2(z23, v2, v3);
                            int q0 = __float2int_rn(__fmul_rn(__fmul_rn(v0, rn.x), rtn));
                            int q1 = __float2int_rn(__fmul_rn(__fmul_rn(v1, rn.y), rtn));
                            int q2 = __float2int_rn(__fmul_rn(__fmul_rn(v2, rn.z), rtn));
                            int q3 = __float2int_rn(__fmul_rn(__fmul_rn(v3, rn.w), rtn));
                            if (p.qmax_next != 127) {
                                q0 = max(min(q0, p.qmax_next), p.qmin_next);
                                q1 = max(min(q1, p.qmax_next), p.qmin_next);
                                q2 = max(min(q2, p.qmax_next), p.qmin_next);
                                q3 = max(min(q3, p.qmax_next), p.qmin_next);
                            }
                            uint32_t hi, packed;
                            asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q3), "r"(q2), "r"(0));
                            asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(packed) : "r"(q1), "r"(q0), "r"(hi));
                            w[h * 8 + j / 4] = packed;
                        }
                    }
                } else if (OUT == STWQ_OUT_BF16) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const uint32_t* r = h == 0 ? r0 : r1;
                            const float4 sw = *reinterpret_cast<const float4*>(csw + h * 32 + j);
                            const float4 bi = *reinterpret_cast<const float4*>(cbi + h * 32 + j);
                            uint64_t z01 = fma_f2(pack_f2((float)(int32_t)r[j + 0], (float)(int32_t)r[j + 1]),
                                                  mul_f2(st2, pack_f2(sw.x, sw.y)), pack_f2(bi.x, bi.y));
                            uint64_t z23 = fma_f2(pack_f2((float)(int32_t)r[j + 2], (float)(int32_t)r[j + 3]),
                                                  mul_f2(st2, pack_f2(sw.z, sw.w)), pack_f2(bi.z, bi.w));
                            z01 = apply_act_f2<ACT>(z01);
                            z23 = apply_act_f2<ACT>(z23);
                            float v0, v1, v2, v3;
                            unpack_f2(z01, v0, v1);
                            unpack_f2(z23, v2, v3);
                            w[h * 16 + j / 2] = pack_bf16(v0, v1);
                            w[h * 16 + j / 2 + 1] = pack_bf16(v2, v3);
                        }
                    }
                } else if (OUT == STWQ_OUT_F32) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const float4 sw = *reinterpret_cast<const float4*>(csw + j);
                        const float4 bi = *reinterpret_cast<const float4*>(cbi + j);
                        const uint64_t z01 = fma_f2(pack_f2((float)(int32_t)r0[j + 0], (float)(int32_t)r0[j + 1]),
                                                    mul_f2(st2, pack_f2(sw.x, sw.y)), pack_f2(bi.x, bi.y));
                        const uint64_t z23 = fma_f2(pack_f2((float)(int32_t)r0[j + 2], (float)(int32_t)r0[j + 3]),
                                                    mul_f2(st2, pack_f2(sw.z, sw.w)), pack_f2(bi.z, bi.w));
                        float v0, v1, v2, v3;
                        unpack_f2(z01, v0, v1);
                        unpack_f2(z23, v2, v3);
                        w[j + 0] = __float_as_uint(apply_act<ACT>(v0));
                        w[j + 1] = __float_as_uint(apply_act<ACT>(v1));
                        w[j + 2] = __float_as_uint(apply_act<ACT>(v2));
                        w[j + 3] = __float_as_uint(apply_act<ACT>(v3));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) w[j] = r0[j];
                }
                if (STORE == 1) {
                    // straight from registers: this thread's 128 contiguous bytes of row `row`
                    if (row < p.M && col0 < p.N) {
                        uint8_t* y = reinterpret_cast<uint8_t*>(p.Y) + ((size_t)grow * (size_t)p.N + (size_t)col0) * kElem;
                        if (p.y_vec32 && col0 + kChunkCols <= p.N) {
#pragma unroll
                            for (int g = 0; g < 4; ++g) st_global_v8(y + g * 32, w + g * 8);
                        } else {
                            const int valid = (p.N - col0) * kElem;        // a multiple of 16 bytes
#pragma unroll
                            for (int g = 0; g < 8; ++g)
                                if (g * 16 < valid) st_global_v4(y + g * 16, w + g * 4);
                        }
                    }
                } else {
                    const uint32_t stage_tile = stage0 + (nstore & 1u) * 4096u;
                    const uint32_t my_row_addr = stage_tile + (uint32_t)lane * 128u;
                    // the store that last used this staging tile (two stores ago) must have been read
                    if (lane == 0) bulk_wait_read1();
                    __syncwarp();
#pragma unroll
                    for (int g = 0; g < 8; ++g) {         // eight 16-byte pieces, swizzled by row
                        const uint32_t piece = (uint32_t)(g ^ (lane & 7));
                        st_shared_v4(my_row_addr + piece * 16u, w[4 * g], w[4 * g + 1], w[4 * g + 2], w[4 * g + 3]);
                    }
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        if (col0 < p.N && (int64_t)m0 + q * 32 < p.M) tma_store_3d(&tmY, stage_tile, col0, m0 + q * 32, g);
                        bulk_commit();    // one group per chunk, even an empty one: wait_group.read 1 counts groups
                    }
                }
            }
        }
        if (STORE == 0 && lane == 0) bulk_wait0();         // stores complete before the CTA may exit
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, STWQ_DEV_TIMEOUT);
    cluster_sync_all();                                  // no remote arrive or multicast still to land
    tc_fence_after();
    if (warp == 2) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * BN) : "memory");
    }
}

// ---------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

}  // namespace

int stwq_encode_2d(stwq_ctx* ctx, CUtensorMap* map, CUtensorMapDataType dt, int elem_bytes, const void* ptr,
                   int64_t rows, int64_t cols, int box_cols, int box_rows)
{
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)cols * (cuuint64_t)elem_bytes};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, dt, 2, const_cast<void*>(ptr), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        ctx->last_cuda_error = (int)r;
        return STWQ_ERR_CUDA;
    }
    return STWQ_OK;
}

int stwq_encode_3d(stwq_ctx* ctx, CUtensorMap* map, CUtensorMapDataType dt, int elem_bytes, const void* ptr,
                   int64_t rows, int64_t cols, int64_t batch, int64_t row_pitch, int64_t batch_pitch, int box_cols,
                   int box_rows)
{
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
    cuuint64_t gdim[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)batch};
    cuuint64_t gstride[2] = {(cuuint64_t)row_pitch, (cuuint64_t)batch_pitch};
    cuuint32_t box[3] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    (void)elem_bytes;
    CUresult r = fn(map, dt, 3, const_cast<void*>(ptr), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        ctx->last_cuda_error = (int)r;
        return STWQ_ERR_CUDA;
    }
    return STWQ_OK;
}

namespace {

template <int BN, int STAGES, int EPI, int OUT, int ACT, int STORE, bool ASYM = false>
int launch_variant(stwq_ctx* ctx, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmY,
                   const Gemm2Params& p, bool dependent, cudaStream_t st)
{
    using L = Smem2<BN, STAGES, EPI, STORE>;
    auto kern = qgemm2_kernel<BN, STAGES, EPI, OUT, ACT, STORE, ASYM>;
    const uint64_t bit = 1ull << ((BN == 256 ? 0 : 16) + OUT * 4 + ACT);
    uint64_t& mask = ctx->configured_pair[STORE + (ASYM ? 2 : 0)];
    if (!(mask & bit)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamic);
        if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
        mask |= bit;
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(64 + 32 * EPI, 1, 1);
    cfg.dynamicSmemBytes = L::kDynamic;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // Persistent kernel with a static tile stride: launch exactly as many CTA pairs as can be
    // resident at once (pairs must sit in one GPC, so this can be fewer than SMs / 2).
    if (ctx->max_pairs <= 0) {
        cfg.gridDim = dim3((unsigned)(ctx->sm_count & ~1), 1, 1);
        int n = 0;
        cudaError_t e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
        if (e != cudaSuccess || n <= 0) return stwq_cuda_fail(ctx, e == cudaSuccess ? cudaErrorLaunchOutOfResources : e);
        ctx->max_pairs = n < ctx->sm_count / 2 ? n : ctx->sm_count / 2;
    }
    int pairs = ctx->max_pairs;
    if (p.num_units < pairs) pairs = p.num_units;
    cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
    cfg.numAttrs = dependent ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmY, p);
    ctx->launches += 1;
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

template <int BN, int STAGES, int EPI, int STORE>
int launch_bn(stwq_ctx* ctx, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmY,
              const Gemm2Params& p, int act, int out_dtype, bool dependent, cudaStream_t st)
{
#define STWQ_CASE(O, A) \
    if (out_dtype == O && act == A) return launch_variant<BN, STAGES, EPI, O, A, STORE>(ctx, tmA, tmB, tmY, p, dependent, st);
    if (p.z_w != nullptr) {                               // asymmetric: staged-store variant of 256-wide tiles only
        if constexpr (BN == 256 && STORE == 0) {
#define STWQ_ACASE(O, A) \
    if (out_dtype == O && act == A) return launch_variant<BN, STAGES, EPI, O, A, STORE, true>(ctx, tmA, tmB, tmY, p, dependent, st);
            if (out_dtype == STWQ_OUT_INT32)
                return launch_variant<BN, STAGES, EPI, STWQ_OUT_INT32, STWQ_ACT_NONE, STORE, true>(ctx, tmA, tmB, tmY, p, dependent, st);
            STWQ_ACASE(STWQ_OUT_F32, STWQ_ACT_NONE)
            STWQ_ACASE(STWQ_OUT_F32, STWQ_ACT_GELU_ERF)
            STWQ_ACASE(STWQ_OUT_F32, STWQ_ACT_GELU_TANH)
            STWQ_ACASE(STWQ_OUT_F32, STWQ_ACT_GELU_FAST)
            STWQ_ACASE(STWQ_OUT_BF16, STWQ_ACT_NONE)
            STWQ_ACASE(STWQ_OUT_BF16, STWQ_ACT_GELU_ERF)
            STWQ_ACASE(STWQ_OUT_BF16, STWQ_ACT_GELU_TANH)
            STWQ_ACASE(STWQ_OUT_BF16, STWQ_ACT_GELU_FAST)
#undef STWQ_ACASE
        }
        return STWQ_ERR_DIM;
    }
    if (out_dtype == STWQ_OUT_INT32)
        return launch_variant<BN, STAGES, EPI, STWQ_OUT_INT32, STWQ_ACT_NONE, STORE>(ctx, tmA, tmB, tmY, p, dependent, st);
    if (out_dtype == kOutCodes) {                         // 128-column chunks: 256-wide tiles only
        if constexpr (BN == 256) {
            STWQ_CASE(kOutCodes, STWQ_ACT_NONE)
            STWQ_CASE(kOutCodes, STWQ_ACT_GELU_ERF)
            STWQ_CASE(kOutCodes, STWQ_ACT_GELU_TANH)
            STWQ_CASE(kOutCodes, STWQ_ACT_GELU_FAST)
        }
        return STWQ_ERR_DIM;
    }
    STWQ_CASE(STWQ_OUT_F32, STWQ_ACT_NONE)
    STWQ_CASE(STWQ_OUT_F32, STWQ_ACT_GELU_ERF)
    STWQ_CASE(STWQ_OUT_F32, STWQ_ACT_GELU_TANH)
    STWQ_CASE(STWQ_OUT_F32, STWQ_ACT_GELU_FAST)
    STWQ_CASE(STWQ_OUT_BF16, STWQ_ACT_NONE)
    STWQ_CASE(STWQ_OUT_BF16, STWQ_ACT_GELU_ERF)
    STWQ_CASE(STWQ_OUT_BF16, STWQ_ACT_GELU_TANH)
    STWQ_CASE(STWQ_OUT_BF16, STWQ_ACT_GELU_FAST)
#undef STWQ_CASE
    return STWQ_ERR_BITS;
}

}  // namespace

// True if the pair kernel can run this problem: TMA needs 16-byte row pitches for Y and the
// epilogue reads s_w / bias as aligned float4.
bool stwq_qgemm2_supported(int N, int out_dtype, const float* s_w, const float* bias)
{
    const int elem = out_dtype == STWQ_OUT_BF16 ? 2 : (out_dtype == kOutCodes ? 1 : 4);
    if (((int64_t)N * elem) % 16 != 0) return false;
    if (out_dtype != STWQ_OUT_INT32) {
        if ((reinterpret_cast<uintptr_t>(s_w) & 15u) != 0) return false;
        if (bias != nullptr && (reinterpret_cast<uintptr_t>(bias) & 15u) != 0) return false;
    }
    return true;
}

int stwq_launch_qgemm2(stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K, int N,
                       const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* bias,
                       int act, int out_dtype, void* Y, bool after_quantize, const stwq_chain* chain, cudaStream_t st,
                       const stwq_asym* asym, const stwq_batch* batch)
{
    const int G = batch ? batch->G : 1;
    // 256-wide tiles whenever N has more than 128 columns: a 128-wide tile needs 1.5x the
    // L2 -> shared-memory bytes per multiply-accumulate and is bound by that feed.
    const int tiles_m = (int)((M + 2 * kBM - 1) / (2 * kBM));
    int bn = (N > 128 || out_dtype == kOutCodes || asym != nullptr) ? 256 : 128;
    if (ctx->force_bn == 128 || ctx->force_bn == 256) bn = ctx->force_bn;

    Gemm2Params p;
    p.z_tok = asym ? asym->z_tok : nullptr;
    p.z_w = asym ? asym->z_w : nullptr;
    p.colsum = asym ? asym->colsum : nullptr;
    p.rowcorr = asym ? asym->rowcorr : nullptr;
    p.Y = Y;
    p.s_ch_next = chain ? chain->s_ch_next : nullptr;
    p.s_tok_next = chain ? chain->s_tok_next : nullptr;
    p.qmax_next = chain ? (1 << (chain->bits_next - 1)) - 1 : 127;
    p.qmin_next = -p.qmax_next - 1;
    if (out_dtype == kOutCodes && (!chain || !chain->s_tok_next)) return STWQ_ERR_NULL;
    const int elem = out_dtype == STWQ_OUT_BF16 ? 2 : (out_dtype == kOutCodes ? 1 : 4);
    p.y_vec32 = ((reinterpret_cast<uintptr_t>(Y) & 31u) == 0 && ((int64_t)N * elem) % 32 == 0) ? 1 : 0;
    p.M = M; p.N = N; p.K = K; p.P = P;
    p.pos_ids = pos_ids; p.s_w = s_w; p.s_tok = s_tok; p.bias = bias;
    p.tiles_n = (N + bn - 1) / bn;
    p.tiles_per_g = tiles_m * p.tiles_n;
    p.num_tiles = G * p.tiles_per_g;
    p.pos_shared = batch ? batch->pos_shared : 1;
    p.sw_gstride = batch ? batch->sw_gstride : 0;
    p.idesc = stwq_ptx::make_idesc_i8(2 * kBM, bn);
    if (batch && batch->a_unsigned) p.idesc &= ~(1u << 7);         // A format field: 0 = unsigned 8-bit
    p.num_kb = (K + kBK - 1) / kBK;
    p.status = ctx->d_status;
    p.wait_limit_ns = (unsigned long long)ctx->wait_limit_ms * 1000000ull;

    // The last wave of a static tile schedule is partly empty unless the tile count divides by
    // the number of pairs. Its tiles can be cut along K into nsplit units each, whose int32
    // partial sums meet in scratch memory (the last unit to arrive adds them up). Measured, this
    // never pays here: each unit writes 256 KB and the last arriver reads them back one after the
    // other at the very end of the kernel, which costs 1 us and more per range (M 4736, N 1024,
    // K 4096, a two-tile tail: 25.6 us whole tiles, 26.9 / 33.0 / 48.4 us with 2 / 4 / 8 ranges),
    // more than the k-blocks saved. So the cut is made only on request (STWQ_OPT_KSPLIT > 0).
    p.full_units = p.num_tiles;
    p.num_units = p.num_tiles;
    p.nsplit = 1;
    p.kb_per_split = p.num_kb;
    p.partial = nullptr;
    p.counters = nullptr;
    const int pairs = ctx->max_pairs > 0 ? ctx->max_pairs : ctx->sm_count / 2;
    const int tail = p.num_tiles % pairs;
    if (bn == 256 && tail > 0 && 2 * tail <= pairs && ctx->force_ksplit > 0 && G == 1) {
        int nsplit = ctx->force_ksplit < p.num_kb ? ctx->force_ksplit : p.num_kb;
        if (nsplit >= 2) {
            const int kbps = (p.num_kb + nsplit - 1) / nsplit;
            nsplit = (p.num_kb + kbps - 1) / kbps;             // every range holds at least one k-block
            const size_t piece_bytes = (size_t)4 * 32 * 32 * sizeof(int32_t);      // 32 rows x 128 columns
            int rc = stwq_split_ws(ctx, (size_t)tail * nsplit * 2 * 8 * piece_bytes, (size_t)tail * 2 * 8, &p.counters,
                                   &p.partial, st);
            if (rc == STWQ_OK && nsplit >= 2) {
                p.full_units = p.num_tiles - tail;
                p.nsplit = nsplit;
                p.kb_per_split = kbps;
                p.num_units = p.full_units + tail * nsplit;
            } else if (rc != STWQ_ERR_DIM) {
                return rc;
            }
        }
    }

    CUtensorMap tmA, tmB, tmY;
    const int64_t ldb = batch ? batch->ldb : K;
    const int64_t bgs = batch ? batch->b_gstride : (int64_t)N * K;
    int rc = stwq_encode_3d(ctx, &tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Xq, M, K, G, K, M * (int64_t)K, kBK, kBM);
    if (rc != STWQ_OK) return rc;
    rc = stwq_encode_3d(ctx, &tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, N, K, G, ldb, bgs, kBK, bn / 2);
    if (rc != STWQ_OK) return rc;
    const int64_t ypitch = (int64_t)N * elem, ygs = M * ypitch;
    if (out_dtype == STWQ_OUT_BF16)
        rc = stwq_encode_3d(ctx, &tmY, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Y, M, N, G, ypitch, ygs, 64, 32);
    else if (out_dtype == STWQ_OUT_F32)
        rc = stwq_encode_3d(ctx, &tmY, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, Y, M, N, G, ypitch, ygs, 32, 32);
    else if (out_dtype == kOutCodes)
        rc = stwq_encode_3d(ctx, &tmY, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Y, M, N, G, ypitch, ygs, 128, 32);
    else
        rc = stwq_encode_3d(ctx, &tmY, CU_TENSOR_MAP_DATA_TYPE_INT32, 4, Y, M, N, G, ypitch, ygs, 32, 32);
    if (rc != STWQ_OK) return rc;
    if (bn == 128) return launch_bn<128, 6, 8, 0>(ctx, tmA, tmB, tmY, p, act, out_dtype, after_quantize, st);
    // Long main loops hide the epilogue anyway and gain from the deeper ring that the
    // register-direct epilogue leaves room for; short ones (and GELU) are bound by the epilogue,
    // which costs the fewest shared-memory cycles when it goes through staged TMA stores.
    // (crossover measured at M 10880, N 1024 and 4096: between K 1536 and 1920 for 2-byte outputs,
    // between 1920 and 2560 for 4-byte ones)
    bool direct = K >= (elem == 4 ? 2304 : 1792) && act == STWQ_ACT_NONE && asym == nullptr;
    if (ctx->debug == 1) direct = false;                  // tuning: force one or the other
    if (ctx->debug == 2 && asym == nullptr) direct = true;
    if (direct) return launch_bn<256, 6, 8, 1>(ctx, tmA, tmB, tmY, p, act, out_dtype, after_quantize, st);
    return launch_bn<256, 4, 8, 0>(ctx, tmA, tmB, tmY, p, act, out_dtype, after_quantize, st);
}
