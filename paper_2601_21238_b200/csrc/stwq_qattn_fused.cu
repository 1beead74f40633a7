// One-kernel quantized attention head (Section 5: the matrix multiplications of attention run in
// 6 or 8 bits, Appendix C: over a quantized KV cache). Same arithmetic as the three separate stages
// (integer Q K^T, fp32 softmax, Eq. 1 quantizer of the probabilities on [0, 1], integer P V, the
// dequantizers of Appendix A.1), but the scores and the probability codes never leave the SM:
//
//   * a CTA owns 128 queries of one head and walks over the visible keys in chunks of 128, handed
//     over in units of 64;
//   * S = Qq Kq^T of a unit: tcgen05.mma kind::i8 (M 128, N 64) into one of 2 to 4 accumulators in
//     tensor memory, operands staged by TMA from the code caches (the head dimension is padded to
//     128 bytes with zeros by TMA). The tensor core runs ahead of the threads by the spare accumulators:
//     from hand-back to a finished MMA it takes about as long as the threads need for a unit;
//   * the probabilities of a row must be divided by the sum over ALL its keys before they can be
//     quantized, so the keys are walked twice: the first walk only keeps the running maximum and
//     the running sum of every row, the second recomputes S, turns it into codes
//     round(p * (2^b - 1)), and writes them into shared memory in the 128-byte-swizzled K-major
//     layout a tensor-core operand needs. Two threads share a row: one takes the first 64 keys of
//     every chunk, the other the second 64, each reading its part of the row from the accumulator;
//     between the walks they exchange their maxima and sums through shared memory;
//   * O += Pcodes (unsigned) x Vq (signed): a second tcgen05.mma per unit (K = 64), accumulated
//     over the chunks in tensor memory, dequantized with delta_p * s_v[c] at the end;
//   * the column scales of the keys (s_kcol) travel with their chunk as a 512-byte bulk copy.
//
// What a thread does per score is ordinary-pipe work except one ex2 per walk: the int32 -> fp32
// conversions are done with the 1.5 * 2^23 trick (|acc| <= 256 * 128 * 128 = 2^22 fits), and so is
// the rounding of the codes; multiplies and adds are packed two to an instruction. The ex2 unit
// (16 results per clock per SM) sets the floor: measured alone, this mix of instructions runs at
// 10 to 11 scores per clock per SM, the whole kernel at about 6. Two CTAs per SM while d <= 128.
//
// HBM traffic: Q codes, the K and V code caches (once per 128 queries, from L2 after the first
// time), and O; against fp32 scores written and read back plus the codes of P in the staged form.
#include <cuda.h>

#include "stwq_internal.cuh"
#include "stwq_ptx.cuh"

using namespace stwq_ptx;

namespace {

constexpr int kQT = 128;          // queries per CTA
constexpr int kKT = 128;          // keys per chunk
constexpr int kMaxStages = 4;     // rings of key and of value chunks: depth chosen per head dimension, at most this
constexpr int kSoftWarps = 8;     // two per tensor-memory lane quarter: one takes the first, one the second 64 keys of every chunk
constexpr int kThreads = 32 * (2 + kSoftWarps);   // warp 0: TMA, warp 1: MMA + tensor memory, then the row threads
constexpr int kTile = 128 * 128;  // bytes of one 128 x 128-byte operand tile
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kMagic = 12582912.0f;             // 1.5 * 2^23: adding it rounds to an integer in the mantissa
constexpr uint32_t kMagicBits = 0x4B400000u;

struct FaParams {
    int Tq, Tk, d, causal, P, n_qt, dkb, out_bf16, kstages, vstages, nbuf;
    const float* Q;               // [G, Tq, d] fp32: quantized by the CTA that owns the rows
    int qmin, qmax;
    const int32_t* pos_q;
    const float* s_q;
    const float* s_kcol;          // padded to a multiple of 128 entries
    const float* s_v;
    float levels;
    void* O;
    uint32_t* status;
    unsigned long long wait_limit_ns;
};

constexpr int kMaxBuf = 4;        // score accumulators of 64 keys in tensor memory
// barriers: q; k and v full / empty per ring stage; sfull, sfree per score accumulator; pfull, pfree per half of
// the code tile; ofull; stats; one per key-scale slot
constexpr int kNumBars = 1 + 4 * kMaxStages + 2 * kMaxBuf + 6 + (kMaxStages + 1);
constexpr int kOffMisc = 384, kOffStats = 512, kOffScales = kOffStats + 2 * 128 * 8;    // relative to the barriers
static_assert(8 * kNumBars <= kOffMisc, "barrier area");

struct FaSmem {
    int offK, offV, offP, offBars, vbytes, total;
    __host__ __device__ FaSmem(int d, int dkb, int kstages, int vstages)
    {
        vbytes = d * 128;                                 // d rows of 128 keys
        offK = dkb * kTile;                               // after the query tile(s)
        offV = offK + kstages * dkb * kTile;
        offP = offV + vstages * vbytes;
        offBars = offP + kTile;
        total = offBars + kOffScales + (kMaxStages + 1) * 512;   // barriers, (max, sum) of both parts of every row, key scales
    }
};


__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}
__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ uint64_t add_f2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
// Two int32 accumulators (|v| <= 2^22) -> fp32, exact, without the conversion unit: the integer added to
// the bit pattern of 1.5 * 2^23 is that float plus the integer.
__device__ __forceinline__ uint64_t acc_to_float2(uint32_t v0, uint32_t v1, uint64_t neg_magic2)
{
    return add_f2(pack_f2(__uint_as_float(v0 + kMagicBits), __uint_as_float(v1 + kMagicBits)), neg_magic2);
}

__global__ void __launch_bounds__(kThreads, 2)
qattn_fused_kernel(const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const FaParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const FaSmem L(p.d, p.dkb, p.kstages, p.vstages);
    const int kKStages = p.kstages, kVStages = p.vstages;

    const uint32_t bars = base + (uint32_t)L.offBars;
    const uint32_t bar_q = bars;
    auto bar_kfull = [&](int s) { return bars + 8u * (1 + s); };
    auto bar_kempty = [&](int s) { return bars + 8u * (1 + kMaxStages + s); };
    auto bar_vfull = [&](int s) { return bars + 8u * (1 + 2 * kMaxStages + s); };
    auto bar_vempty = [&](int s) { return bars + 8u * (1 + 3 * kMaxStages + s); };
    // the 128 keys of a chunk are handed over in two halves of 64, each with its own four barriers
    const uint32_t bar_half = bars + 8u * (1 + 4 * kMaxStages);
    auto bar_sfull = [&](int b) { return bar_half + 8u * b; };
    auto bar_sfree = [&](int b) { return bar_half + 8u * (kMaxBuf + b); };
    auto bar_pfull = [&](int h) { return bar_half + 8u * (2 * kMaxBuf + h); };
    auto bar_pfree = [&](int h) { return bar_half + 8u * (2 * kMaxBuf + 2 + h); };
    const uint32_t bar_ofull = bar_half + 8u * (2 * kMaxBuf + 4);
    const uint32_t bar_stats = bar_half + 8u * (2 * kMaxBuf + 5);
    // The column scales of a chunk of keys travel with the chunk (512 bytes, a bulk copy), but live
    // longer than its ring stage: the row threads still read them after the score MMAs are done. A
    // stage is freed by the second score MMA of a chunk, which was issued after the row threads handed
    // back the buffer of nbuf units earlier; with nbuf <= 4 that leaves at most the chunk before it in
    // the row threads' hands, so two slots more than stages are enough.
    auto bar_cfull = [&](int c) { return bar_half + 8u * (2 * kMaxBuf + 6 + c); };
    const int cslots = kKStages + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L.offBars + kOffMisc);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // long (late) query tiles first: under a causal mask they walk over the most keys
    const int qt = p.n_qt - 1 - (int)blockIdx.y;
    const int g = blockIdx.x;
    const int q0 = qt * kQT;
    const int kmax = p.causal ? min(p.Tk - 1, min(q0 + kQT - 1, p.Tq - 1) + p.Tk - p.Tq) : p.Tk - 1;   // last key any row sees
    const int nch = kmax / kKT + 1;
    const int nbuf = p.nbuf;                             // score accumulators: columns 64 b .. 64 b + 63
    const int tmem_cols = p.d <= 128 ? 256 : 512;        // O follows them: columns 64 nbuf .. 64 nbuf + d - 1

    if (threadIdx.x == 0) {
        mbar_init(bar_q, kSoftWarps);                     // the row threads write the query codes
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(bar_kfull(s), 1);
            mbar_init(bar_kempty(s), 1);
            mbar_init(bar_vfull(s), 1);
            mbar_init(bar_vempty(s), 1);
        }
        for (int b = 0; b < kMaxBuf; ++b) {
            mbar_init(bar_sfull(b), 1);
            mbar_init(bar_sfree(b), kSoftWarps / 2);     // a unit belongs to one of the two groups of row threads
        }
        for (int h = 0; h < 2; ++h) {
            mbar_init(bar_pfull(h), kSoftWarps / 2);
            mbar_init(bar_pfree(h), 1);
        }
        mbar_init(bar_ofull, 1);
        mbar_init(bar_stats, kSoftWarps);
        for (int c = 0; c <= kMaxStages; ++c) mbar_init(bar_cfull(c), 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        tc_fence_before();
    }
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const unsigned long long limit = p.wait_limit_ns;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // One thread feeds both rings and never blocks on one of them while the other could take a
        // load: the value chunks of the second walk start arriving during the first.
        if (lane == 0) {
            int ik = 0, iv = 0;                           // next key load (of 2 nch), next value load (of nch)
            bool ok = true;
            unsigned long long t0 = globaltimer_ns();
            uint32_t polls = 0;
            while (ik < 2 * nch || iv < nch) {
                bool progressed = false;
                if (ik < 2 * nch) {
                    const int s = ik % kKStages;
                    if (mbar_try_wait(bar_kempty(s), ((uint32_t)(ik / kKStages) & 1u) ^ 1u)) {
                        const int j = ik < nch ? ik : ik - nch;
                        mbar_expect_tx(bar_kfull(s), (uint32_t)(p.dkb * kTile));
                        for (int kb = 0; kb < p.dkb; ++kb)
                            tma_load_3d(base + L.offK + (s * p.dkb + kb) * kTile, &tmK, kb * 128, j * kKT, g, bar_kfull(s));
                        const int c = ik % cslots;
                        mbar_expect_tx(bar_cfull(c), 512u);
                        bulk_load(base + (uint32_t)(L.offBars + kOffScales + c * 512), p.s_kcol + j * kKT, 512u, bar_cfull(c));
                        ++ik;
                        progressed = true;
                    }
                }
                if (iv < nch) {
                    const int sv = iv % kVStages;
                    if (mbar_try_wait(bar_vempty(sv), ((uint32_t)(iv / kVStages) & 1u) ^ 1u)) {
                        mbar_expect_tx(bar_vfull(sv), (uint32_t)L.vbytes);
                        tma_load_3d(base + L.offV + sv * L.vbytes, &tmV, iv * kKT, 0, g, bar_vfull(sv));
                        ++iv;
                        progressed = true;
                    }
                }
                if (progressed) {
                    t0 = globaltimer_ns();
                    continue;
                }
                __nanosleep(100);                         // leave the issue slots to the row threads
                if ((++polls & 31u) == 0u) {
                    if (*abort_flag) { ok = false; break; }
                    if (globaltimer_ns() - t0 > limit) { *abort_flag = 1u; ok = false; break; }
                }
            }
            if (!ok) {
                // giving up: loads already issued may still be landing in this CTA's shared memory
                t0 = globaltimer_ns();
                for (int b = 1; b <= kKStages && ik - b >= 0; ++b) {
                    const int jt = ik - b;
                    while (!mbar_try_wait(bar_kfull(jt % kKStages), (uint32_t)(jt / kKStages) & 1u))
                        if (globaltimer_ns() - t0 > limit) break;
                }
                for (int b = 1; b <= cslots && ik - b >= 0; ++b) {
                    const int jt = ik - b;
                    while (!mbar_try_wait(bar_cfull(jt % cslots), (uint32_t)(jt / cslots) & 1u))
                        if (globaltimer_ns() - t0 > limit) break;
                }
                for (int b = 1; b <= kVStages && iv - b >= 0; ++b) {
                    const int jv = iv - b;
                    while (!mbar_try_wait(bar_vfull(jv % kVStages), (uint32_t)(jv / kVStages) & 1u))
                        if (globaltimer_ns() - t0 > limit) break;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // The unit of work is half a chunk: 64 keys. Unit u = 2 * (chunk visit) + half goes into score
        // accumulator u % nbuf, so the tensor core runs up to nbuf - 1 units ahead of the row
        // threads (issue, execution and the wake-up through the barrier take longer than the rows
        // need for a unit). The P V product of a unit is issued behind the score MMA of the next one.
        if (lane == 0) {
            const uint32_t idesc_s = make_idesc_i8(kQT, kKT / 2);
            const uint32_t idesc_pv = make_idesc_i8(kQT, p.d) & ~(1u << 7);      // A = unsigned codes
            const uint32_t tmem_o = tmem_base + 64u * nbuf;
            bool ok = mbar_wait(bar_q, 0u, abort_flag, limit);
            auto issue_pv = [&](int u) -> bool {                                  // unit u of the second walk
                const int j = u / 2 - nch, h = u & 1;
                const int sv = j % kVStages;
                if (h == 0 && !mbar_wait(bar_vfull(sv), (uint32_t)(j / kVStages) & 1u, abort_flag, limit)) return false;
                if (!mbar_wait(bar_pfull(h), (uint32_t)j & 1u, abort_flag, limit)) return false;
                tc_fence_after();
                const uint64_t a_desc = make_smem_desc(base + L.offP) + 4u * h;   // 64 bytes further along the keys
                const uint64_t b_desc = make_smem_desc(base + L.offV + sv * L.vbytes) + 4u * h;
#pragma unroll
                for (int k = 0; k < 2; ++k)
                    tc_mma_i8(tmem_o, a_desc + 2u * k, b_desc + 2u * k, idesc_pv, (j | h | k) != 0 ? 1u : 0u);
                tc_commit(bar_pfree(h));
                if (h == 1) tc_commit(bar_vempty(sv));
                return true;
            };
            const int units = 4 * nch;
            int b = 0;                                    // score accumulator of unit u: u % nbuf
            uint32_t free_parity = 0u;                    // parity of the hand-back of the buffer's previous use
            for (int u = 0; ok && u < units; ++u) {
                const int it = u >> 1, h = u & 1;
                const int s = it % kKStages;
                if (h == 0 && !mbar_wait(bar_kfull(s), (uint32_t)(it / kKStages) & 1u, abort_flag, limit)) { ok = false; break; }
                if (u >= nbuf && !mbar_wait(bar_sfree(b), free_parity, abort_flag, limit)) { ok = false; break; }
                tc_fence_after();
                for (int kb = 0; kb < p.dkb; ++kb) {
                    const uint64_t a_desc = make_smem_desc(base + kb * kTile);
                    const uint64_t b_desc = make_smem_desc(base + L.offK + (s * p.dkb + kb) * kTile + h * (kTile / 2));
                    const int nk = min(4, (p.d - kb * 128 + 31) / 32);           // the rest of the 128 bytes is TMA's zero fill
                    for (int k = 0; k < nk; ++k)
                        tc_mma_i8(tmem_base + 64u * b, a_desc + 2u * k, b_desc + 2u * k, idesc_s, (kb | k) != 0 ? 1u : 0u);
                }
                tc_commit(bar_sfull(b));
                if (h == 1) tc_commit(bar_kempty(s));
                if (++b == nbuf) {
                    b = 0;
                    if (u >= nbuf) free_parity ^= 1u;
                }
                if (u - 1 >= 2 * nch && !issue_pv(u - 1)) { ok = false; break; }
            }
            if (ok) ok = issue_pv(units - 1);
            if (ok) tc_commit(bar_ofull);
        }
    } else {
        // ------------------------------------------------------------------ two threads per query row
        // Warps 2..5 take the first 64 keys of every chunk (the even units), warps 6..9 the second 64
        // (the odd units): two independent streams of work per row, each with its own score
        // accumulators in flight. A row's maximum and sum are therefore kept in two parts, which the
        // two threads exchange through shared memory between the walks.
        // Per score and walk: one integer add and half a packed add (conversion), half a packed
        // multiply (column scale), half a packed fma (row scale, minus the maximum), one ex2; the
        // first walk adds half a 3-input max and half a packed add, the second half a packed fma
        // (scale to codes and round) and three quarters of a byte permute.
        const int h = (warp - 2) >> 2;                    // which half of every chunk
        // The queries of this tile -> codes (the static per-position quantizer: (x * 1) * (1 / s_q[pos]),
        // round to nearest even, clamp), written as the A operand: rows of 128 bytes, 16-byte pieces
        // swizzled by the row, zeros beyond the head dimension. A thread takes 16 consecutive
        // channels at a time; consecutive threads walk along the row.
        {
            const int rt_id = (int)threadIdx.x - 64;      // 0 .. 255
            const int pieces = p.dkb * 8;                 // 16-byte pieces per row, over all 128-byte blocks
            const int live = p.d >> 4;                    // pieces that hold channels
            for (int t = rt_id; t < kQT * pieces; t += kSoftWarps * 32) {
                const int row = t / pieces, c16 = t - row * pieces;
                const int qi = q0 + row;
                uint32_t w[4] = {0u, 0u, 0u, 0u};
                if (c16 < live && qi < p.Tq) {
                    const int pos = p.pos_q[qi];
                    if (pos >= 0 && pos < p.P) {
                        const float rt = __frcp_rn(p.s_q[pos]);
                        const float4* src = reinterpret_cast<const float4*>(p.Q + ((int64_t)g * p.Tq + qi) * p.d) + c16 * 4;
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const float4 x = __ldg(src + k);
                            const int c0 = stwq_code(__fmul_rn(x.x, rt), p.qmin, p.qmax), c1 = stwq_code(__fmul_rn(x.y, rt), p.qmin, p.qmax);
                            const int c2 = stwq_code(__fmul_rn(x.z, rt), p.qmin, p.qmax), c3 = stwq_code(__fmul_rn(x.w, rt), p.qmin, p.qmax);
                            w[k] = (uint32_t)(c0 & 0xFF) | ((uint32_t)(c1 & 0xFF) << 8) | ((uint32_t)(c2 & 0xFF) << 16) | ((uint32_t)(c3 & 0xFF) << 24);
                        }
                    }
                }
                const int kb = c16 >> 3, piece = c16 & 7;
                st_shared_v4(base + (uint32_t)(kb * kTile) + (uint32_t)(row >> 3) * 1024u + (uint32_t)(row & 7) * 128u +
                                 (uint32_t)((piece ^ (row & 7)) * 16),
                             w[0], w[1], w[2], w[3]);
            }
            fence_async_smem();                           // the codes become visible to the tensor core's reads
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_q);
        }
        const int q = warp & 3;                           // the lane quarter of tensor memory this warp may read
        const int r = q * 32 + lane;                      // row of the tile
        const int i = q0 + r;                             // query index within the head
        const bool valid = i < p.Tq;
        float a = 0.0f;
        if (valid) {
            const int pos = p.pos_q[i];
            if (pos >= 0 && pos < p.P) a = p.s_q[pos];
            else if (g == 0 && h == 0) atomicOr(p.status, STWQ_DEV_POS_RANGE);
        }
        // rows beyond Tq see no key at all: a warp of such rows skips every block (and still hands the
        // accumulators back and writes zero codes); in a mixed warp they run along, masked, and are not stored
        const int last = !valid ? -1 : (p.causal ? min(p.Tk - 1, i + p.Tk - p.Tq) : p.Tk - 1);   // last visible key of the row
        const int wlast = __reduce_max_sync(0xffffffffu, last);
        const int wfirst = __reduce_min_sync(0xffffffffu, last);
        const float al = fmaxf(a * kLog2e, 1e-30f);       // scores are kept in units of log2 e; > 0 so that a masked -inf stays -inf
        const uint64_t al2 = dup_f2(al);
        const uint64_t neg_magic2 = dup_f2(-kMagic);
        const uint64_t magic2 = dup_f2(kMagic);
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t prow = base + (uint32_t)L.offP + (uint32_t)(r >> 3) * 1024u + (uint32_t)(r & 7) * 128u;
        const uint8_t* scales = smem + L.offBars + kOffScales;
        float2* stats = reinterpret_cast<float2*>(smem + L.offBars + kOffStats);     // [2][128]: (max, sum) of each part
        float m = -INFINITY, l = 0.0f;
        uint64_t inv2 = 0;
        int b = h % nbuf, cslot = 0;                      // unit u = 2 it + h lives in accumulator u % nbuf
        uint32_t sparity = 0u, cparity = 0u;
        bool ok = true;
        for (int it = 0; ok && it < 2 * nch; ++it) {
            const bool second = it >= nch;
            const int j = second ? it - nch : it;
            if (it == nch) {
                // both parts of the row: m = max of the two, l = the two sums brought to that maximum
                stats[h * 128 + r] = make_float2(m, l);
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_stats);
                ok = mbar_wait(bar_stats, 0u, abort_flag, limit);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const float2 other = stats[(h ^ 1) * 128 + r];
                const float mt = fmaxf(m, other.x);      // finite for every row below Tq: the first part has seen key 0
                const float rt = mt == -INFINITY ? 0.0f : mt;
                l = l * ex2f(m - rt) + other.y * ex2f(other.x - rt);
                m = rt;                                   // a row beyond Tq: every key masked, codes 0
                inv2 = dup_f2(l > 0.0f ? __fdiv_rn(p.levels, l) : 0.0f);      // l = 0: a row beyond Tq
            }
            {
                ok = mbar_wait(bar_cfull(cslot), cparity, abort_flag, limit);
                if (ok) ok = mbar_wait(bar_sfull(b), sparity, abort_flag, limit);
                if (ok && second && j > 0) ok = mbar_wait(bar_pfree(h), (uint32_t)(j - 1) & 1u, abort_flag, limit);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
#pragma unroll 1
                for (int blk = 0; blk < 2; ++blk) {
                    const int cb = 2 * h + blk;           // 32-key block of the chunk
                    const int col0 = j * kKT + cb * 32;
                    const uint32_t pc0 = prow + (uint32_t)(((2 * cb) ^ (r & 7)) * 16);
                    const uint32_t pc1 = prow + (uint32_t)(((2 * cb + 1) ^ (r & 7)) * 16);
                    if (col0 > wlast) {                   // nobody in this warp sees these keys
                        if (second) {
                            st_shared_v4(pc0, 0u, 0u, 0u, 0u);
                            st_shared_v4(pc1, 0u, 0u, 0u, 0u);
                        }
                        continue;
                    }
                    uint32_t v[32];
                    tmem_ld32(taddr + (uint32_t)(b * 64 + blk * 32), v);
                    tmem_ld_wait();
                    const float4* kc = reinterpret_cast<const float4*>(scales + cslot * 512) + cb * 8;
                    const bool cut = col0 + 31 > wfirst;  // the mask cuts through this block for some row
                    // y = acc * s_kcol; the score in units of log2 e is y * (s_q * log2 e)
                    uint64_t y2[16];
#pragma unroll
                    for (int c = 0; c < 16; c += 2) {
                        const float4 s4 = kc[c >> 1];
                        y2[c] = mul_f2(acc_to_float2(v[2 * c], v[2 * c + 1], neg_magic2), pack_f2(s4.x, s4.y));
                        y2[c + 1] = mul_f2(acc_to_float2(v[2 * c + 2], v[2 * c + 3], neg_magic2), pack_f2(s4.z, s4.w));
                    }
                    if (cut) {
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            float y0, y1;
                            unpack_f2(y2[c], y0, y1);
                            if (col0 + 2 * c > last) y0 = -INFINITY;
                            if (col0 + 2 * c + 1 > last) y1 = -INFINITY;
                            y2[c] = pack_f2(y0, y1);
                        }
                    }
                    if (!second) {
                        // maximum as a tree of 3-input operations, sums in four packed partial sums: a
                        // chain of dependent operations would be paid in full with so few warps
                        float pm[8];
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            float y0, y1, y2a, y3;
                            unpack_f2(y2[c], y0, y1);
                            unpack_f2(y2[c + 8], y2a, y3);
                            pm[c] = fmaxf(max3(y0, y1, y2a), y3);
                        }
                        const float bm = max3(max3(pm[0], pm[1], pm[2]), max3(pm[3], pm[4], pm[5]), fmaxf(pm[6], pm[7]));
                        const float mn = fmaxf(m, bm * al);          // -inf only while the row has seen no key (never after block 0)
                        const float ref = mn == -INFINITY ? 0.0f : mn;
                        const uint64_t nref2 = dup_f2(-ref);
                        uint64_t ps[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            float t0, t1;
                            unpack_f2(fma_f2(y2[c], al2, nref2), t0, t1);
                            ps[c & 3] = add_f2(ps[c & 3], pack_f2(ex2f(t0), ex2f(t1)));
                        }
                        float s0, s1;
                        unpack_f2(add_f2(add_f2(ps[0], ps[1]), add_f2(ps[2], ps[3])), s0, s1);
                        l = l * ex2f(m - ref) + (s0 + s1);
                        m = mn;
                    } else {
                        const uint64_t nm2 = dup_f2(-m);
                        uint32_t w[8];
#pragma unroll
                        for (int c = 0; c < 16; c += 2) {
                            float t0, t1, t2, t3;
                            unpack_f2(fma_f2(y2[c], al2, nm2), t0, t1);
                            unpack_f2(fma_f2(y2[c + 1], al2, nm2), t2, t3);
                            // u = p * levels; adding 1.5 * 2^23 leaves round-to-nearest-even(u) in the low mantissa bits
                            const uint64_t u01 = fma_f2(pack_f2(ex2f(t0), ex2f(t1)), inv2, magic2);
                            const uint64_t u23 = fma_f2(pack_f2(ex2f(t2), ex2f(t3)), inv2, magic2);
                            w[c >> 1] = prmt(prmt((uint32_t)u01, (uint32_t)(u01 >> 32), 0x0040u),
                                             prmt((uint32_t)u23, (uint32_t)(u23 >> 32), 0x0040u), 0x5410u);
                        }
                        st_shared_v4(pc0, w[0], w[1], w[2], w[3]);
                        st_shared_v4(pc1, w[4], w[5], w[6], w[7]);
                    }
                }
                tc_fence_before();
                if (second) fence_async_smem();           // the codes become visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) {
                    if (second) mbar_arrive(bar_pfull(h));
                    mbar_arrive(bar_sfree(b));
                }
                b += 2;
                if (b >= nbuf) {
                    b -= nbuf;
                    sparity ^= 1u;
                }
            }
            if (++cslot == cslots) {
                cslot = 0;
                cparity ^= 1u;
            }
        }
        // ------------------------------------------------------------------ O = acc * (delta_p * s_v[c])
        if (ok) ok = mbar_wait(bar_ofull, 0u, abort_flag, limit);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc_fence_after();
            const float delta_p = __fdiv_rn(1.0f, p.levels);
            const int64_t row_off = ((int64_t)g * p.Tq + i) * p.d;
#pragma unroll 1
            for (int cb = h; cb * 32 < p.d; cb += 2) {   // the two threads of a row take alternate 32-column blocks
                uint32_t v[32];
                tmem_ld32(taddr + (uint32_t)(64 * nbuf + cb * 32), v);
                tmem_ld_wait();
                const int ncol = min(32, p.d - cb * 32);  // 32 or 16
                const float4* sv4 = reinterpret_cast<const float4*>(p.s_v + cb * 32);
                float o[32];
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (c < ncol) s4 = __ldg(sv4 + (c >> 2));
                    o[c] = __fmul_rn((float)(int32_t)v[c], __fmul_rn(delta_p, s4.x));
                    o[c + 1] = __fmul_rn((float)(int32_t)v[c + 1], __fmul_rn(delta_p, s4.y));
                    o[c + 2] = __fmul_rn((float)(int32_t)v[c + 2], __fmul_rn(delta_p, s4.z));
                    o[c + 3] = __fmul_rn((float)(int32_t)v[c + 3], __fmul_rn(delta_p, s4.w));
                }
                if (valid) {
                    if (p.out_bf16) {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.O) + row_off + cb * 32);
#pragma unroll
                        for (int c = 0; c < 32; c += 8)
                            if (c < ncol)
                                dst[c >> 3] = make_uint4(pack_bf16(o[c], o[c + 1]), pack_bf16(o[c + 2], o[c + 3]),
                                                         pack_bf16(o[c + 4], o[c + 5]), pack_bf16(o[c + 6], o[c + 7]));
                    } else {
                        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.O) + row_off + cb * 32);
#pragma unroll
                        for (int c = 0; c < 32; c += 4)
                            if (c < ncol) dst[c >> 2] = make_float4(o[c], o[c + 1], o[c + 2], o[c + 3]);
                    }
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, STWQ_DEV_TIMEOUT);
    tc_fence_after();
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

}  // namespace

// Q [G, Tq, d] fp32 queries; Kc [G, Tmax, d], Vt [G, d, Tmax] the code caches; s_kcol_pad
// holds at least round_up(Tk, 128) entries. O [G, Tq, d] fp32 or bf16.
int stwq_launch_qattn_fused(stwq_ctx* ctx, const float* Q, const int32_t* pos_q, int G, int Tq, int Tk, int d, int Tmax,
                            const int8_t* Kc, const int8_t* Vt, const float* s_q, const float* s_kcol_pad, const float* s_v,
                            int P, int bits, int causal, int out_dtype, void* O, cudaStream_t st)
{
    FaParams p;
    p.Tq = Tq; p.Tk = Tk; p.d = d; p.causal = causal ? 1 : 0; p.P = P;
    p.n_qt = (Tq + kQT - 1) / kQT;
    p.dkb = (d + 127) / 128;
    p.out_bf16 = out_dtype == STWQ_OUT_BF16 ? 1 : 0;
    p.Q = Q;
    p.qmax = (1 << (bits - 1)) - 1;
    p.qmin = -(1 << (bits - 1));
    p.pos_q = pos_q; p.s_q = s_q; p.s_kcol = s_kcol_pad; p.s_v = s_v;
    p.levels = (float)((1 << bits) - 1);
    p.O = O;
    p.status = ctx->d_status;
    p.wait_limit_ns = (unsigned long long)ctx->wait_limit_ms * 1000000ull;
    CUtensorMap tmK, tmV;
    int rc = stwq_encode_3d(ctx, &tmK, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Kc, Tmax, d, G, d, (int64_t)Tmax * d, 128, kKT);
    if (rc != STWQ_OK) return rc;
    rc = stwq_encode_3d(ctx, &tmV, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Vt, d, Tmax, G, Tmax, (int64_t)d * Tmax, kKT, d);
    if (rc != STWQ_OK) return rc;
    if (p.n_qt > 65535) return STWQ_ERR_DIM;
    // ring depths: as deep as two CTAs per SM allow (113 KB each) while d <= 128; beyond that a CTA
    // holds all 512 columns of tensor memory and the SM to itself
    p.kstages = d <= 64 ? 3 : (d <= 128 ? 2 : 3);
    p.vstages = d <= 64 ? 3 : 2;
    // score accumulators of 64 columns beside the d columns of O: 256 columns of tensor memory per CTA while d <= 128
    p.nbuf = d <= 64 ? 3 : (d <= 128 ? 2 : 4);
    static_assert(3 + 2 <= kMaxStages + 1 && 4 <= kMaxBuf, "key-scale slots: two more than the deepest key ring");
    const FaSmem L(d, p.dkb, p.kstages, p.vstages);
    int dyn = L.total + 1024;
    if (dyn < 78 * 1024) dyn = 78 * 1024;
    if (!ctx->attn_configured) {
        cudaError_t e = cudaFuncSetAttribute(qattn_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024);
        if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
        ctx->attn_configured = 1;
    }
    qattn_fused_kernel<<<dim3((unsigned)G, (unsigned)p.n_qt), kThreads, (size_t)dyn, st>>>(tmK, tmV, p);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}
