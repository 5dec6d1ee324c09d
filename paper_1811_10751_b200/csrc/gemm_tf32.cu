// FP32-storage worker products (steps O1, O2) and coded update (O3) on the 5th-generation tensor
// cores: tcgen05.mma kind::tf32 with the accumulator in tensor memory, operands brought into
// shared memory by TMA, and 3xTF32 splitting so that the result keeps FP32-level accuracy:
//     a = a_hi + a_lo (both exactly representable in TF32),   a*b ~ a_lo*b_hi + a_hi*b_lo + a_hi*b_hi.
//
// One CTA per SM walks a list of 128 x 128 tiles of the nodes' products.  The tiles left over after
// the last full round over the SMs are cut into pieces that fit one more, short round: products into
// parts of their contraction, whose sums meet in a scratch buffer of the plan (a part costs its share
// of a tile's time, where a column strip still pays for all of A: cut into four strips, 24 left-over
// tiles of the 4096 x 4096 layer cost 0.73 of a full round, cut into six parts 0.4); the update, whose
// output is read-modify-write, into column strips.
//
// Accumulation.  The tensor cores add into their FP32 accumulator with truncation, so a long chain
// of MMAs loses up to one ulp of the running sum per step, always towards zero: over K = 2048
// (768 steps) that is 1.4e-5 of the output's rms, which a threshold-9 decoder amplifies beyond
// the 1e-4 bar.  The chain is therefore kept short: tensor memory only holds the partial sum of
// group_kb k-blocks (one k-block: K = 32, 12 steps).  Two accumulators in tensor memory alternate
// between groups; the eight warps that split the operands also pull every finished partial sum
// into FP32 registers (each owns a lane quarter and half of the columns: 64 values per thread)
// and add the groups up with round-to-nearest.  At a tile's end they write the sums back into
// the accumulator they drained last, from where the four epilogue warps take them while the next
// tile's main loop is already running.
// Warp roles:
//   warp 0       : TMA producer (one lane) - raw FP32 tiles of A and B into a 4-stage ring that
//                  runs on across tiles
//   warp 1       : allocates tensor memory; one lane issues the MMAs of the even k-blocks and commits them
//                  to mbarriers (the last warp's lane 0 does the same for the odd k-blocks)
//   warps 2..9   : split every landed pair of tiles: B in place in shared memory (hi overwrites the
//                  raw tile, lo goes to a second tile); A row by row into tensor memory (hi and lo, 32
//                  columns each per stage), from where the MMAs take it: the A operand then costs
//                  shared-memory bandwidth once (its raw read) instead of four times.  Two k-blocks
//                  behind their conversions they drain the finished accumulation groups (above)
//   warps 10..13 : read a finished tile back (tcgen05.ld), hand the accumulator back to the MMA
//                  warp, and write the tile (plain store, or read-modify-write for the coded update)
// Operand tiles use the 128-byte swizzle; A is K-major; B is K-major for the update (X^_p is
// [N][K]) and MN-major for the forward / backward products (X~_p, W~_p are [K][N]).
// Tensor memory (512 columns): accumulators in columns 0..255, the A stages behind them.
// Every mbarrier wait is bounded; on expiry the CTA raises a status word, drains its copies,
// frees its tensor memory and returns.
#include <cuda.h>

#include <type_traits>

#include "gemm_common.h"
#include "tc_common.h"

namespace gpd {

namespace {

constexpr int BM = 128, BN = 128, BK = 32, STAGES = 4;
constexpr int UMMA_K = 8;
constexpr int A_TILE_BYTES = BM * BK * 4;            // 16 KB, rows of 128 B
constexpr int B_TILE_BYTES = BN * BK * 4;            // 16 KB
constexpr int STAGE_BYTES = A_TILE_BYTES + 2 * B_TILE_BYTES;   // raw A, B hi, B lo
// k-blocks whose products are summed in tensor memory before they move to registers.  Measured error
// of a product (K = 2048, against an FP64 product of the same shares, relative to the output's rms):
// 2.8e-7 for groups of one k-block, 4.7e-7 for two, 9.1e-7 for four, 1.8e-6 for eight, 1.4e-5 with no
// cut at all.  Decoding amplifies it: at threshold 9 the worst threshold-sized subset of 11 nodes
// turns 2.8e-7 into 2.7e-5 of relative Frobenius error (an ideal FP32 product: 2e-5).  Products
// decoded with a threshold of 7 or more use groups of one k-block, smaller thresholds two.  The
// update contracts over the mini-batch only and its result is a small increment of the share, so
// one chain of up to 256 elements is accurate enough there and keeps a whole tile of lead for the
// read-modify-write.
constexpr int kGroupKbProduct = 2, kGroupKbProductLarge = 1, kGroupKbUpdate = 8;
constexpr int kDrainLag = 2;                         // update kernel: a group is drained this many conversions after its last k-block
constexpr int kEpiWarps = 4;                         // update kernel, warps 10..13: drain a finished tile, one per lane quarter
constexpr int EPI_PITCH = 36;                        // floats per staged row: 16-byte aligned, conflict-free for 16-byte accesses
constexpr int kEpiWarpsD = 8;                        // product kernel, warps 10..17: drain every group (64 columns of a lane quarter each)
constexpr int EPI_COLS_D = 16;                       // product kernel: columns of a staged chunk
constexpr int EPI_PITCH_D = 20;
constexpr int EPI_STAGE_BYTES = kEpiWarpsD * 32 * EPI_PITCH_D * 4;   // one 32 x 16 chunk per warp (update kernel: 32 x 32 for four warps fits too)
static_assert(kEpiWarps * 32 * EPI_PITCH * 4 <= EPI_STAGE_BYTES, "staging area of the update kernel");
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_STAGE_BYTES + 1024;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
constexpr int TMEM_ACC_COLS = 2 * BN;                // two 128-column accumulators: one fills while the other drains
constexpr int TMEM_A_COLS = 2 * BK;                  // per stage: A hi (BK columns), A lo (BK columns); lane = row of the tile
constexpr int TMEM_COLS = 512;
static_assert(TMEM_ACC_COLS + STAGES * TMEM_A_COLS <= TMEM_COLS, "tensor memory budget");
constexpr int kConvWarps = 8;                        // warps 2..9: split tiles
constexpr int kConvThreads = kConvWarps * 32;
// Who adds the groups up: the product kernel has eight epilogue warps for it (18 warps, 96 registers a
// thread); the update kernel, which has one group per tile for mini-batches up to 256 and whose
// read-modify-write epilogue wants wide chunks and a whole tile of lead, lets the splitting warps do
// it (14 warps, 128 registers).  Measured on 10 x [2048 x 2048] x [2048 x 256]: products 0.178 ms with
// the first arrangement and 0.207 ms with the second; update 0.217 ms and 0.147 ms.
template <bool UPDATE> constexpr int kThreadsOf = 64 + kConvThreads + (UPDATE ? kEpiWarps : kEpiWarpsD) * 32 + 32;   // + second issuer

__device__ int g_tf32_status = 0;                    // GPD_ERR_TIMEOUT if a bounded wait expired

using tc::kWaitCycles;
using tc::mbar_arrive;
using tc::mbar_expect_tx;
using tc::mbar_init;
using tc::mbar_try_wait;
using tc::smem_u32;
using tc::tma_load_3d;
using tc::umma_commit;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    return tc::mbar_wait(bar, parity, abort_flag, &g_tf32_status);
}
// Hand-over between the two MMA issuers: a counter in shared memory, written with release and read with
// acquire semantics.  The wait is bounded like the barrier waits.
__device__ __forceinline__ bool turn_wait(int* turn, int want, volatile int* abort_flag) {
    const long long t0 = clock64();
    for (;;) {
        int v;
        asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(turn)) : "memory");
        if (v >= want) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            atomicExch(&g_tf32_status, (int)GPD_ERR_TIMEOUT);
            return false;
        }
    }
}
__device__ __forceinline__ void turn_pass(int* turn, int next) {
    asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32(turn)), "r"(next) : "memory");
}
// for the epilogue warps: they wait most of the time, and a poll every 200 ns is early enough for them
__device__ __forceinline__ bool mbar_wait_relaxed(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    return tc::mbar_wait(bar, parity, abort_flag, &g_tf32_status, kWaitCycles, 200);
}

// Shared-memory matrix descriptor: start address, leading / stride byte offsets in 16-byte units,
// descriptor version 1, layout type (2 = 128-byte swizzle of 16-byte chunks, used for K-major
// operands; 1 = 128-byte swizzle of 32-byte chunks, the only layout an MN-major 32-bit operand
// may use).
constexpr uint32_t kLayoutSw128 = 2, kLayoutSw128Base32 = 1;
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)layout << 61;
    return d;
}
// K-major tile: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t addr) { return smem_desc(addr, 16, 1024, kLayoutSw128); }
// MN-major tile: [k][32 columns] rows of 128 bytes; 4-row swizzle groups 512 bytes apart (two per
// MMA of K = 8); the next 32 columns start BK rows (BK * 128 bytes) further.
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr) { return smem_desc(addr, BK * 128, 512, kLayoutSw128Base32); }

// A operand from tensor memory (lane = row, one column per TF32 element)
__device__ __forceinline__ void umma_tf32_ta(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// 16 consecutive columns of this thread's lane
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}

// Round to the nearest TF32 value (10 explicit mantissa bits) with integer arithmetic: add half
// a TF32 ulp to the magnitude and clear the 13 low bits (ties away from zero; Inf stays Inf).
__device__ __forceinline__ float to_tf32(float x) {
    return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u);
}

// What the tensor core makes of a raw FP32 word in a TF32 operand: the 13 low mantissa bits dropped.
__device__ __forceinline__ float trunc_tf32(float x) { return __uint_as_float(__float_as_uint(x) & 0xFFFFE000u); }

// Split contraction, after a warp has written its 32 x 64 piece of one part's sum into the scratch
// buffer: the warp takes a ticket on the piece; the warps with the same index in the other parts' CTAs
// do the same.  Whoever draws the last ticket adds the parts up in the order of the parts (so the sum
// does not depend on who came last) and stores the piece into C.  Kept out of line: it runs once per
// left-over tile and must not cost the main loop registers.
__device__ __noinline__ void splitk_finish(const float* kscratch, unsigned int* kcount, int left, int ksplit, int ew,
                                           float* Cg, int64_t M, int64_t N, int m0, int n0) {
    const int lane = threadIdx.x & 31;
    const int q = (threadIdx.x >> 5) & 3, ch = (ew >> 2) * (BN / 2);
    const int col4 = (lane & 3) * 4, rsub = lane >> 2;
    __threadfence();
    __syncwarp();
    unsigned int ticket = 0;
    if (lane == 0) ticket = atomicAdd(&kcount[left * kEpiWarpsD + ew], 1u);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    if (ticket != (unsigned int)(ksplit - 1)) return;            // another part will finish this piece
    __threadfence();
    const float* parts = kscratch + (size_t)left * ksplit * (size_t)(BM * BN);
    const bool vec_c = (N % 4 == 0);
#pragma unroll 1
    for (int c0 = 0; c0 < BN / 2; c0 += EPI_COLS_D) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = q * 32 + 8 * i + rsub, col = ch + c0 + col4;
            float4 sum = __ldcg(reinterpret_cast<const float4*>(parts + (size_t)row * BN + col));
            for (int pp = 1; pp < ksplit; ++pp) {
                const float4 v = __ldcg(reinterpret_cast<const float4*>(parts + (size_t)pp * (BM * BN) + (size_t)row * BN + col));
                sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
            }
            const int64_t grow = (int64_t)m0 + row, gcol = (int64_t)n0 + col;
            if (grow < M) {
                float* dst = Cg + grow * N + gcol;
                if (vec_c && gcol + 4 <= N) {
                    *reinterpret_cast<float4*>(dst) = sum;
                } else {
                    if (gcol < N) dst[0] = sum.x;
                    if (gcol + 1 < N) dst[1] = sum.y;
                    if (gcol + 2 < N) dst[2] = sum.z;
                    if (gcol + 3 < N) dst[3] = sum.w;
                }
            }
        }
    }
}

// KSPLIT: the instantiation that cuts left-over tiles along the contraction (products only; launched
// only when there is something to cut, so that the plain walk over whole tiles keeps its registers).
template <bool B_KMAJOR, bool UPDATE, bool KSPLIT>
__global__ void __launch_bounds__(kThreadsOf<UPDATE>, 1)
sgemm_3xtf32_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmParams prm,
                    int tiles_m, int tiles_n, int full_tiles, int split, int ksplit, int n_virtual, int group_kb,
                    float* kscratch, unsigned int* kcount) {
    if (UPDATE && prm.gate && prm.gate->outcome == GPD_DECODE_FAILURE) return;
    constexpr bool EPI_DRAINS = !UPDATE;             // the epilogue warps (not the splitting warps) add the groups up
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    // full / conv / empty: operand ring, runs on across the tiles of this CTA; acc_full[b] / acc_empty[b]:
    // accumulator b (tensor-memory columns 128 b ..) complete / read back
    // tile_full[t & 1]: tile t's sums are back in tensor memory (written by the eight splitting warps); two
    // barriers, because tile t + 1 (the other accumulator) can be complete before the epilogue warps, still
    // storing tile t - 1, start to wait for tile t
    __shared__ __align__(8) uint64_t full_bar[STAGES], conv_bar[STAGES], empty_bar[STAGES], acc_full[2], acc_empty[2], tile_full[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int issue_turn;                       // index of the k-block whose MMAs may be issued next

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kIssuer2Warp = kThreadsOf<UPDATE> / 32 - 1;   // the last warp: second MMA issuer
    const int num_kb = (int)((prm.K + BK - 1) / BK);
    // Virtual tile list: whole 128 x 128 tiles first; the tiles left over after the last full round
    // over the SMs follow in pieces, so that the last, partly filled round is short.  Products
    // (ksplit > 1): `ksplit` parts of the contraction each - a part costs its share of a tile's time;
    // the parts' sums meet in a scratch buffer and the last part to arrive adds them up in the order
    // of the parts.  Update (split > 1): `split` column strips each (128 x 32 strips when split = 4;
    // a strip still pays for all of A, so the gain is smaller).  CTA b takes virtual tiles b, b + grid, ...
    // kb0, nkb: the piece's k-blocks; part: its index among the tile's parts; left: index of the
    // left-over tile (-1 for a whole tile or a strip).
    auto decode_k = [&](int vt, int& p, int& m0, int& n0, int& bn, int& kb0, int& nkb, int& part, int& left) {
        int tile = vt, sub = 0;
        bn = BN; kb0 = 0; nkb = num_kb; part = 0; left = -1;
        if (vt >= full_tiles) {
            const int piece = vt - full_tiles;
            if (KSPLIT) {
                left = piece / ksplit;
                part = piece - left * ksplit;
                tile = full_tiles + left;
                kb0 = (int)((long long)part * num_kb / ksplit);
                nkb = (int)((long long)(part + 1) * num_kb / ksplit) - kb0;
            } else {
                tile = full_tiles + piece / split;
                sub = piece % split;
                bn = BN / split;
            }
        }
        const int tn = tile % tiles_n, tm = (tile / tiles_n) % tiles_m;
        p = tile / (tiles_n * tiles_m);
        m0 = tm * BM;
        n0 = tn * BN + sub * bn;
    };
    auto decode = [&](int vt, int& p, int& m0, int& n0, int& bn) {
        int tile = vt, sub = 0;
        bn = BN;
        if (vt >= full_tiles) {
            const int piece = vt - full_tiles;
            tile = full_tiles + piece / split;
            sub = piece % split;
            bn = BN / split;
        }
        const int tn = tile % tiles_n, tm = (tile / tiles_n) % tiles_m;
        p = tile / (tiles_n * tiles_m);
        m0 = tm * BM;
        n0 = tn * BN + sub * bn;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&conv_bar[s], kConvWarps);
            mbar_init(&empty_bar[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1);
            // a group's accumulator is handed back by the eight splitting warps, a tile's last one by
            // the four epilogue warps arriving twice each
            mbar_init(&acc_empty[b], kConvWarps);
        }
        mbar_init(&tile_full[0], kConvWarps);
        mbar_init(&tile_full[1], kConvWarps);
        abort_flag = 0;
        issue_turn = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_slot;
    volatile int* abort_p = &abort_flag;

    auto A_raw = [&](int s) { return smem + s * STAGE_BYTES; };
    auto B_hi = [&](int s) { return smem + s * STAGE_BYTES + A_TILE_BYTES; };
    auto B_lo = [&](int s) { return smem + s * STAGE_BYTES + A_TILE_BYTES + B_TILE_BYTES; };
    auto A_tmem = [&](int s) { return tmem_base + (uint32_t)(TMEM_ACC_COLS + s * TMEM_A_COLS); };   // hi; lo is BK columns further

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            int it = 0;                          // k-blocks issued so far, over all tiles
            bool ok = true;
            for (int vt = blockIdx.x; vt < n_virtual && ok; vt += gridDim.x) {
                int p, m0, n0, bn, kb0 = 0, nkb = num_kb, part = 0, left = -1;
                if constexpr (KSPLIT) decode_k(vt, p, m0, n0, bn, kb0, nkb, part, left);
                else decode(vt, p, m0, n0, bn);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    const int k0 = (kb0 + kb) * BK;
                    if (!mbar_wait(&empty_bar[s], ph ^ 1, abort_p)) { ok = false; break; }
                    mbar_expect_tx(&full_bar[s], A_TILE_BYTES + bn * BK * 4);
                    tma_load_3d(A_raw(s), &tmA, k0, m0, p, &full_bar[s]);
                    for (int c = 0; c < bn / 32; ++c) {      // B arrives in boxes of 32 columns (or 32 rows of X^_p)
                        if (B_KMAJOR)
                            tma_load_3d(B_hi(s) + c * (BK * 128), &tmB, k0, n0 + 32 * c, p, &full_bar[s]);
                        else
                            tma_load_3d(B_hi(s) + c * (BK * 128), &tmB, n0 + 32 * c, k0, p, &full_bar[s]);
                    }
                }
            }
            if (*abort_p) {                      // let copies still in flight land before the CTA exits
                for (int j = it > STAGES ? it - STAGES : 0; j < it; ++j) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(&full_bar[j % STAGES], (j / STAGES) & 1) && clock64() - t0 < kWaitCycles) {}
                }
            }
        }
    } else if (warp == 1 || warp == kIssuer2Warp) {
        // ------------------------------ MMA issuers ------------------------------
        // Two threads take the k-blocks in turn (lane 0 of warp 1 the even ones, lane 0 of the last warp
        // the odd ones).  Everything a k-block needs besides the MMAs themselves - waiting for its operands
        // and for a free accumulator, building descriptors, committing to the barriers afterwards - costs
        // a single thread as many cycles as issuing the twelve MMAs does (issue blocks while the tensor
        // pipe is busy; measured 700 cycles of issue and 700-900 of the rest per k-block), and the pipe's
        // queue is too short to bridge that.  With two issuers one thread's bookkeeping runs under the
        // other's MMAs; only the hand-over (a release / acquire on a shared-memory counter, with the
        // tcgen05 fences that order the two threads' MMAs) lies between the k-blocks.
        if (lane == 0) {
            const int me = warp == 1 ? 0 : 1;
            int it = 0, gi = 0;                   // k-blocks / accumulation groups so far, over all tiles (both issuers count alike)
            bool ok = true;
            for (int vt = blockIdx.x; vt < n_virtual && ok; vt += gridDim.x) {
                int p, m0, n0, bn, kb0 = 0, nkb = num_kb, part = 0, left = -1;
                if constexpr (KSPLIT) decode_k(vt, p, m0, n0, bn, kb0, nkb, part, left);
                else decode(vt, p, m0, n0, bn);
                const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((B_KMAJOR ? 0u : 1u) << 16) |
                                       ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
                int kg = 0;                      // position of the k-block inside its accumulation group
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int buf = gi & 1;
                    const bool group_end = kg == group_kb - 1 || kb == nkb - 1;
                    if ((it & 1) == me) {
                        if (kg == 0) {
                            // the group before last used this accumulator: it must have been read back
                            if (!mbar_wait(&acc_empty[buf], ((gi >> 1) & 1) ^ 1, abort_p)) { ok = false; break; }
                        }
                        const uint32_t tmem_d = tmem_base + (uint32_t)(buf * BN);
                        const int s = it % STAGES;
                        const uint32_t ph = (it / STAGES) & 1;
                        if (!mbar_wait(&conv_bar[s], ph, abort_p)) { ok = false; break; }
                        // the two B descriptors are built once per stage, a k-step only adds its offset to
                        // their address field (16-byte units, no carry out of 14 bits: a stage lies inside
                        // the 227 KB window)
                        const uint32_t a_hi = A_tmem(s), a_lo = A_tmem(s) + BK;
                        const uint64_t db_hi0 = B_KMAJOR ? desc_kmajor(smem_u32(B_hi(s))) : desc_mnmajor(smem_u32(B_hi(s)));
                        const uint64_t db_lo0 = db_hi0 + (uint64_t)(B_TILE_BYTES >> 4);
                        // my turn: the other issuer has handed over after its last MMA of k-block it - 1
                        if (!turn_wait(&issue_turn, it, abort_p)) { ok = false; break; }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k) {
                            // A: the next 8 elements of K are 8 tensor-memory columns further.
                            // B, K-major: 32 bytes further inside the swizzled row; MN-major: the next 8
                            // k-rows are 8 * 128 bytes further in every 32-column chunk
                            const uint32_t a_off = k * UMMA_K;
                            const uint64_t b_off = (uint64_t)((B_KMAJOR ? k * UMMA_K * 4 : k * UMMA_K * 128) >> 4);
                            const uint32_t first = (kg > 0 || k > 0) ? 1u : 0u;    // a group starts from zero
                            umma_tf32_ta(tmem_d, a_lo + a_off, db_hi0 + b_off, idesc, first);   // small terms first
                            umma_tf32_ta(tmem_d, a_hi + a_off, db_lo0 + b_off, idesc, 1u);
                            umma_tf32_ta(tmem_d, a_hi + a_off, db_hi0 + b_off, idesc, 1u);
                        }
                        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                        turn_pass(&issue_turn, it + 1);
                        umma_commit(&empty_bar[s]);      // stage reusable once these MMAs have read it
                        // this group's partial sum complete: the group's earlier MMAs (the other issuer's
                        // among them) feed the same accumulator, so they have finished when these have
                        if (group_end) umma_commit(&acc_full[buf]);
                    }
                    if (group_end) { ++gi; kg = 0; } else { ++kg; }
                }
            }
        }
    } else if (warp < 2 + kConvWarps) {
        // ------------------------------ split hi / lo, drain groups ------------------------------
        const int tc = threadIdx.x - 64;             // 0..kConvThreads-1
        // A: this warp may touch tensor-memory lanes 32 q .. 32 q + 31 (q = warp mod 4); the two warps
        // of a quarter take 16 of the 32 k-columns each.  A thread owns one row of the tile.
        const int q = warp & 3, khalf = (warp - 2) >> 2;
        const int arow = q * 32 + lane;
        // Accumulation groups: this warp adds up columns 64 khalf .. 64 khalf + 63 of its lane quarter.
        const int n_groups = (num_kb + group_kb - 1) / group_kb;
        int n_tiles_mine = 0;
        for (int vt = blockIdx.x; vt < n_virtual; vt += gridDim.x) ++n_tiles_mine;
        const int total_groups = n_tiles_mine * n_groups;
        float acc[BN / 2];
        int drained = 0;                             // groups drained so far, over all tiles
        // index (over all tiles of this CTA) of the last k-block of group g
        auto last_kblock = [&](int g) {
            const int t = g / n_groups, j = g - t * n_groups;
            return t * num_kb + min((j + 1) * group_kb, num_kb) - 1;
        };
        // Pull group g's partial sum into the registers; after a tile's last group write the sums back.
        auto drain = [&](int g) -> bool {
            const int t = g / n_groups, j = g - t * n_groups, buf = g & 1;
            int p, m0, n0, bn;
            decode(blockIdx.x + t * (int)gridDim.x, p, m0, n0, bn);
            const bool ready = mbar_wait(&acc_full[buf], (g >> 1) & 1, abort_p);
            __syncwarp();
            if (!__all_sync(0xffffffffu, ready)) return false;   // tcgen05.ld is warp-collective: all lanes or none
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + khalf * (BN / 2));
#pragma unroll
            for (int c = 0; c < BN / 2; c += 32) {
                if (khalf * (BN / 2) + c < bn) {     // strips are 64 or 32 columns wide
                    uint32_t r[32];
                    asm volatile(
                        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                        : "r"(tbase + (uint32_t)c));
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        acc[c + i] = j == 0 ? __uint_as_float(r[i]) : acc[c + i] + __uint_as_float(r[i]);
                }
            }
            if (j < n_groups - 1) {                  // hand the accumulator back to the MMA warp
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[buf]);
                return true;
            }
            // the tile is complete: its sums go back into the accumulator just read, for the epilogue warps
#pragma unroll
            for (int c = 0; c < BN / 2; c += 16) {
                if (khalf * (BN / 2) + c < bn) {
                    uint32_t r[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(acc[c + i]);
                    tmem_st16(tbase + (uint32_t)c, r);
                }
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&tile_full[t & 1]);
            return true;
        };
        int it = 0;
        bool ok = true;
        for (int vt = blockIdx.x; vt < n_virtual && ok; vt += gridDim.x) {
            int p, m0, n0, bn, kb0 = 0, nkb = num_kb, part = 0, left = -1;
            if constexpr (KSPLIT) decode_k(vt, p, m0, n0, bn, kb0, nkb, part, left);
            else decode(vt, p, m0, n0, bn);
            const int b_float4 = bn * BK / 4;        // 16-byte units of one B tile
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1;
                const bool landed = mbar_wait(&full_bar[s], ph, abort_p);
                __syncwarp();
                if (!__all_sync(0xffffffffu, landed)) { ok = false; break; }   // tcgen05.st is warp-collective: all lanes or none
                {   // A row: four 16-byte chunks of the 128-byte swizzled row (chunk index xor row mod 8)
                    const uint8_t* rowp = A_raw(s) + arow * 128;
                    uint32_t hi[16], lo[16];
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const float4 v = *reinterpret_cast<const float4*>(rowp + (((khalf * 4 + c) ^ (arow & 7)) << 4));
                        const float h0 = to_tf32(v.x), h1 = to_tf32(v.y), h2 = to_tf32(v.z), h3 = to_tf32(v.w);
                        hi[4 * c] = __float_as_uint(h0); hi[4 * c + 1] = __float_as_uint(h1);
                        hi[4 * c + 2] = __float_as_uint(h2); hi[4 * c + 3] = __float_as_uint(h3);
                        lo[4 * c] = __float_as_uint(to_tf32(v.x - h0)); lo[4 * c + 1] = __float_as_uint(to_tf32(v.y - h1));
                        lo[4 * c + 2] = __float_as_uint(to_tf32(v.z - h2)); lo[4 * c + 3] = __float_as_uint(to_tf32(v.w - h3));
                    }
                    const uint32_t taddr = A_tmem(s) + ((uint32_t)(q * 32) << 16) + (uint32_t)(khalf * 16);
                    tmem_st16(taddr, hi);
                    tmem_st16(taddr + BK, lo);
                }
                {   // B in place
                    float4* hi = reinterpret_cast<float4*>(B_hi(s));
                    float4* lo = reinterpret_cast<float4*>(B_lo(s));
#pragma unroll 4
                    for (int idx = tc; idx < b_float4; idx += kConvThreads) {
                        const float4 v = hi[idx];
                        float4 l;
                        l.x = to_tf32(v.x - trunc_tf32(v.x)); l.y = to_tf32(v.y - trunc_tf32(v.y));
                        l.z = to_tf32(v.z - trunc_tf32(v.z)); l.w = to_tf32(v.w - trunc_tf32(v.w));
                        lo[idx] = l;
                    }
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");       // A is in tensor memory
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // B tiles visible to the MMA unit
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(&conv_bar[s]);
                // groups whose last k-block was converted kDrainLag conversions ago: their MMAs have
                // (nearly) finished, so the wait inside drain() is short
                if constexpr (!EPI_DRAINS) {
                    while (ok && drained < total_groups && it >= last_kblock(drained) + kDrainLag) ok = drain(drained++);
                    if (!ok) break;
                }
            }
        }
        if constexpr (!EPI_DRAINS) {
            while (ok && drained < total_groups) ok = drain(drained++);   // what the lag left over
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        if constexpr (EPI_DRAINS) {
            // products: eight warps (lane quarter = warp mod 4, column half = (warp - 10) / 4) pull every
            // finished group into registers, add the groups up and store the tile at its end
            const int ew = warp - (2 + kConvWarps);      // 0..7
            const int q = warp & 3;                      // this warp may touch TMEM lanes 32q .. 32q+31
            const int ch = (ew >> 2) * (BN / 2);         // first of this warp's 64 columns of the tile
            [[maybe_unused]] const float shrink = (float)prm.shrink, eta = (float)prm.eta;
            [[maybe_unused]] const bool vec = (prm.N % 4 == 0);
            float* st = reinterpret_cast<float*>(smem + STAGES * STAGE_BYTES) + ew * (32 * EPI_PITCH_D);
            const int col4 = (lane & 3) * 4, rsub = lane >> 2;    // this lane's part of a staged 32 x 16 chunk
            int gi = 0;
            bool ok = true;
            for (int vt = blockIdx.x; vt < n_virtual && ok; vt += gridDim.x) {
                int p, m0, n0, bn, kb0 = 0, nkb = num_kb, part = 0, left = -1;
                if constexpr (KSPLIT) decode_k(vt, p, m0, n0, bn, kb0, nkb, part, left);
                else decode(vt, p, m0, n0, bn);
                const int n_groups = (nkb + group_kb - 1) / group_kb;
                float acc[BN / 2];                       // this thread's row, this warp's columns
                for (int g = 0; g < n_groups; ++g, ++gi) {
                    const int buf = gi & 1;
                    const bool acc_ready = mbar_wait_relaxed(&acc_full[buf], (gi >> 1) & 1, abort_p);
                    __syncwarp();
                    if (!__all_sync(0xffffffffu, acc_ready)) { ok = false; break; }   // tcgen05.ld is warp-collective: all lanes or none
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    #pragma unroll
                    for (int c = 0; c < BN / 2; c += 16) {
                        if (ch + c < bn) {               // strips are 64 or 32 columns wide
                            uint32_t r[16];
                            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + ch + c);
                            asm volatile(
                                "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                                "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                                : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                                  "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                                : "r"(taddr));
                            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
    #pragma unroll
                            for (int j = 0; j < 16; ++j)
                                acc[c + j] = g == 0 ? __uint_as_float(r[j]) : acc[c + j] + __uint_as_float(r[j]);
                        }
                    }
                    // this group's partial sum is in registers: hand the accumulator back
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[buf]);
                }
                if (!ok) break;
                if constexpr (!KSPLIT) {
                    const int64_t gm = (int64_t)m0 + q * 32 + lane;
                    float* C = reinterpret_cast<float*>(prm.C) + (int64_t)p * prm.M * prm.N;
    #pragma unroll
                    for (int c0 = 0; c0 < BN / 2; c0 += EPI_COLS_D) {
                        if (ch + c0 >= bn) break;
                        const int64_t gc = (int64_t)n0 + ch + c0;           // first global column of the chunk
                        const bool whole = vec && gc + EPI_COLS_D <= prm.N;
                        if (whole) {
                            // A thread holds the columns of one row; written as they are, a store would touch 32
                            // rows with 16 bytes each.  A 32 x 16 chunk goes through shared memory instead and
                            // leaves as 64-byte row segments (four lanes per row, eight rows per store).  The
                            // update asks for the stored share before it stages the chunk.
                            float4 old[4];
                            if (UPDATE) {
    #pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const int64_t grow = (int64_t)m0 + q * 32 + 8 * i + rsub;
                                    old[i] = grow < prm.M ? *reinterpret_cast<const float4*>(C + grow * prm.N + gc + col4)
                                                          : make_float4(0.f, 0.f, 0.f, 0.f);
                                }
                            }
    #pragma unroll
                            for (int j = 0; j < EPI_COLS_D; j += 4)
                                *reinterpret_cast<float4*>(st + lane * EPI_PITCH_D + j) =
                                    make_float4(acc[c0 + j], acc[c0 + j + 1], acc[c0 + j + 2], acc[c0 + j + 3]);
                            __syncwarp();
    #pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int row = 8 * i + rsub;
                                const int64_t grow = (int64_t)m0 + q * 32 + row;
                                float4 v = *reinterpret_cast<const float4*>(st + row * EPI_PITCH_D + col4);
                                if (grow < prm.M) {
                                    if (UPDATE) {
                                        const float4 o = old[i];
                                        v.x = shrink * o.x + eta * v.x; v.y = shrink * o.y + eta * v.y;
                                        v.z = shrink * o.z + eta * v.z; v.w = shrink * o.w + eta * v.w;
                                    }
                                    *reinterpret_cast<float4*>(C + grow * prm.N + gc + col4) = v;
                                }
                            }
                            __syncwarp();                        // the next chunk reuses the staging rows
                        } else if (gm < prm.M) {
                            float* crow = C + gm * prm.N + gc;
    #pragma unroll
                            for (int j = 0; j < EPI_COLS_D; ++j) {
                                if (gc + j < prm.N) {
                                    float v = acc[c0 + j];
                                    if (UPDATE) v = shrink * crow[j] + eta * v;
                                    crow[j] = v;
                                }
                            }
                        }
                    }
                } else {
                    // Where the tile goes: into C, or - one part of a left-over tile's contraction - into that
                    // part's 128 x 128 slot of the scratch buffer (same code; base, pitch and limits are
                    // compile-time constants there).
                    auto store_tile = [&](auto part_tag) {
                        constexpr bool PART = decltype(part_tag)::value;
                        float* C = PART ? kscratch + ((size_t)left * ksplit + part) * (size_t)(BM * BN)
                                        : reinterpret_cast<float*>(prm.C) + (int64_t)p * prm.M * prm.N;
                        const int64_t ldc = PART ? BN : prm.N, row_lim = PART ? BM : prm.M, col_lim = PART ? BN : prm.N;
                        const int64_t row0 = PART ? 0 : m0, col0 = PART ? 0 : n0;
                        const bool vec = (ldc % 4 == 0);
                        const int64_t gm = row0 + q * 32 + lane;
    #pragma unroll
                        for (int c0 = 0; c0 < BN / 2; c0 += EPI_COLS_D) {
                            if (ch + c0 >= bn) break;
                            const int64_t gc = col0 + ch + c0;                  // first column of the chunk
                            const bool whole = vec && gc + EPI_COLS_D <= col_lim;
                            if (whole) {
                                // A thread holds the columns of one row; written as they are, a store would touch
                                // 32 rows with 16 bytes each.  A 32 x 16 chunk goes through shared memory instead
                                // and leaves as 64-byte row segments (four lanes per row, eight rows per store).
    #pragma unroll
                                for (int j = 0; j < EPI_COLS_D; j += 4)
                                    *reinterpret_cast<float4*>(st + lane * EPI_PITCH_D + j) =
                                        make_float4(acc[c0 + j], acc[c0 + j + 1], acc[c0 + j + 2], acc[c0 + j + 3]);
                                __syncwarp();
    #pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const int row = 8 * i + rsub;
                                    const int64_t grow = row0 + q * 32 + row;
                                    const float4 v = *reinterpret_cast<const float4*>(st + row * EPI_PITCH_D + col4);
                                    if (grow < row_lim) *reinterpret_cast<float4*>(C + grow * ldc + gc + col4) = v;
                                }
                                __syncwarp();                        // the next chunk reuses the staging rows
                            } else if (gm < row_lim) {
                                float* crow = C + gm * ldc + gc;
    #pragma unroll
                                for (int j = 0; j < EPI_COLS_D; ++j)
                                    if (gc + j < col_lim) crow[j] = acc[c0 + j];
                            }
                        }
                    };
                    if (left < 0) {
                        store_tile(std::false_type{});
                    } else {
                        store_tile(std::true_type{});
                        splitk_finish(kscratch, kcount, left, ksplit, ew, reinterpret_cast<float*>(prm.C) + (int64_t)p * prm.M * prm.N,
                                      prm.M, prm.N, m0, n0);
                    }
                }
            }
        } else {
            // update: four warps read a finished tile back from tensor memory and apply it to the shares
            const int q = warp & 3;                      // this warp may touch TMEM lanes 32q .. 32q+31
            const float shrink = (float)prm.shrink, eta = (float)prm.eta;
            const bool vec = (prm.N % 4 == 0);
            const int n_groups = (num_kb + group_kb - 1) / group_kb;
            int ti = 0;
            for (int vt = blockIdx.x; vt < n_virtual; vt += gridDim.x, ++ti) {
                int p, m0, n0, bn;
                decode(vt, p, m0, n0, bn);
                const int buf = ((ti + 1) * n_groups - 1) & 1;      // the accumulator of the tile's last group holds its sums
                const bool tile_ready = mbar_wait_relaxed(&tile_full[ti & 1], (ti >> 1) & 1, abort_p);
                __syncwarp();
                if (!__all_sync(0xffffffffu, tile_ready)) break;   // tcgen05.ld is warp-collective: all lanes or none
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const int64_t gm = (int64_t)m0 + q * 32 + lane;
                float* C = reinterpret_cast<float*>(prm.C) + (int64_t)p * prm.M * prm.N;
    #pragma unroll 1
                for (int c0 = 0; c0 < bn; c0 += 32) {
                    const bool whole = vec && n0 + c0 + 32 <= prm.N;     // the chunk leaves as 128-byte row segments
                    const int col4 = (lane & 7) * 4, rsub = lane >> 3;   // this lane's part of a staged chunk
                    float4 old[8];                                       // the stored share, asked for before the accumulator is read
                    if (UPDATE && whole) {
    #pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int64_t grow = (int64_t)m0 + q * 32 + 4 * i + rsub;
                            old[i] = grow < prm.M ? *reinterpret_cast<const float4*>(C + grow * prm.N + n0 + c0 + col4)
                                                  : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
                    }
                    uint32_t r[32];
                    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c0);
                    asm volatile(
                        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                        : "r"(taddr));
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (c0 + 32 >= bn) {                 // last read of this accumulator: hand it back (two arrivals per warp)
                        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                        __syncwarp();
                        if (lane == 0) { mbar_arrive(&acc_empty[buf]); mbar_arrive(&acc_empty[buf]); }
                    }
                    if (whole) {
                        // A thread holds 32 columns of one row; written as they are, a store would touch 32
                        // rows with 16 bytes each.  The chunk goes through shared memory instead and
                        // leaves as whole 128-byte row segments (eight lanes per row, four rows per store).
                        float* st = reinterpret_cast<float*>(smem + STAGES * STAGE_BYTES) + (warp - 2 - kConvWarps) * (32 * EPI_PITCH);
    #pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<float4*>(st + lane * EPI_PITCH + j) =
                                make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]),
                                            __uint_as_float(r[j + 3]));
                        __syncwarp();
    #pragma unroll
                        for (int rr = 0; rr < 32; rr += 4) {
                            const int row = rr + rsub;
                            const int64_t grow = (int64_t)m0 + q * 32 + row;
                            float4 v = *reinterpret_cast<const float4*>(st + row * EPI_PITCH + col4);
                            if (grow < prm.M) {
                                float* cp = C + grow * prm.N + n0 + c0 + col4;
                                if (UPDATE) {
                                    const float4 o = old[rr / 4];
                                    v.x = shrink * o.x + eta * v.x; v.y = shrink * o.y + eta * v.y;
                                    v.z = shrink * o.z + eta * v.z; v.w = shrink * o.w + eta * v.w;
                                }
                                *reinterpret_cast<float4*>(cp) = v;
                            }
                        }
                        __syncwarp();                        // the next chunk reuses the staging rows
                    } else if (gm < prm.M) {
                        float* crow = C + gm * prm.N + n0 + c0;
    #pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (n0 + c0 + j < prm.N) {
                                float v = __uint_as_float(r[j]);
                                if (UPDATE) v = shrink * crow[j] + eta * v;
                                crow[j] = v;
                            }
                        }
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---- host side -------------------------------------------------------------------------------------
// 3-D FP32 tensor [batch][rows][cols] (cols contiguous), box {box_cols, box_rows, 1}, given
// 128-byte swizzle flavour, out-of-range elements read as zero.
bool make_map(CUtensorMap* map, const void* base, int64_t batch, int64_t rows, int64_t cols, int box_cols, int box_rows,
              CUtensorMapSwizzle swizzle) {
    return tc::make_map_3d(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, base, batch, rows, cols, box_cols, box_rows, swizzle);
}

// Scratch of the split contraction: counters of `rem` left-over tiles, then `pieces` part sums of one tile each.
constexpr int64_t kSplitKHeaderBytes(int64_t rem) { return (rem * kEpiWarpsD * (int64_t)sizeof(unsigned int) + 255) / 256 * 256; }

template <bool B_KMAJOR, bool UPDATE>
gpd_status launch(const GemmParams& prm, cudaStream_t st) {
    CUtensorMap tmA, tmB;
    if (!make_map(&tmA, prm.A, prm.P, prm.M, prm.K, BK, BM, CU_TENSOR_MAP_SWIZZLE_128B)) return GPD_ERR_CUDA;
    const bool okB = B_KMAJOR ? make_map(&tmB, prm.B, prm.P, prm.N, prm.K, BK, 32, CU_TENSOR_MAP_SWIZZLE_128B)
                              : make_map(&tmB, prm.B, prm.P, prm.K, prm.N, 32, BK, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B);
    if (!okB) return GPD_ERR_CUDA;
    if (cudaFuncSetAttribute(sgemm_3xtf32_kernel<B_KMAJOR, UPDATE, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(sgemm_3xtf32_kernel<B_KMAJOR, UPDATE, !UPDATE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             SMEM_BYTES) != cudaSuccess)
        return GPD_ERR_CUDA;
    const int tiles_n = (int)((prm.N + BN - 1) / BN), tiles_m = (int)((prm.M + BM - 1) / BM);
    const int64_t tiles = (int64_t)tiles_n * tiles_m * prm.P;
    // One CTA per SM at a time.  After the last full round, `rem` tiles are left.  Products: each is cut
    // into as many parts of its contraction as still fit in one round (at least four k-blocks per part),
    // if the caller gave a scratch buffer for the parts' sums.  Otherwise (and for the update, whose
    // output is read-modify-write): 2 or 4 column strips each, if the strips still fit in one round.
    const int sms = sm_count();
    const int rem = (int)(tiles % sms);
    const int num_kb = (int)((prm.K + BK - 1) / BK);
    int split = 1, ksplit = 1;
    if (!UPDATE && rem > 0 && prm.splitk_scratch) {
        ksplit = std::min(std::min(sms / rem, num_kb / 4), 32);
        while (ksplit > 1 && sgemm_3xtf32_scratch_bytes(rem * ksplit) > prm.splitk_bytes) --ksplit;
        if (ksplit < 2) ksplit = 1;
    }
    if (ksplit == 1) {
        if (rem > 0 && rem * 4 <= sms) split = 4;
        else if (rem > 0 && rem * 2 <= sms) split = 2;
    }
    const int pieces = ksplit > 1 ? ksplit : split;
    const int full_tiles = (int)(tiles - (pieces > 1 ? rem : 0));
    const int64_t n_virtual = full_tiles + (int64_t)(pieces > 1 ? rem : 0) * pieces;
    const unsigned grid = (unsigned)std::min<int64_t>(n_virtual, sms);   // persistent: one CTA per SM walks the list
    const int group_kb = UPDATE ? kGroupKbUpdate : (prm.max_threshold >= 7 ? kGroupKbProductLarge : kGroupKbProduct);
    float* kscratch = nullptr;
    unsigned int* kcount = nullptr;
    if (ksplit > 1) {
        // counters first (one per left-over tile and epilogue warp), the parts' sums 256 bytes further on
        kcount = reinterpret_cast<unsigned int*>(prm.splitk_scratch);
        kscratch = reinterpret_cast<float*>(reinterpret_cast<char*>(prm.splitk_scratch) + kSplitKHeaderBytes(rem));
        if (cudaMemsetAsync(kcount, 0, sizeof(unsigned int) * rem * kEpiWarpsD, st) != cudaSuccess) return GPD_ERR_CUDA;
    }
    if (ksplit > 1)
        sgemm_3xtf32_kernel<B_KMAJOR, UPDATE, !UPDATE><<<grid, kThreadsOf<UPDATE>, SMEM_BYTES, st>>>(
            tmA, tmB, prm, tiles_m, tiles_n, full_tiles, split, ksplit, (int)n_virtual, group_kb, kscratch, kcount);
    else
        sgemm_3xtf32_kernel<B_KMAJOR, UPDATE, false><<<grid, kThreadsOf<UPDATE>, SMEM_BYTES, st>>>(
            tmA, tmB, prm, tiles_m, tiles_n, full_tiles, split, ksplit, (int)n_virtual, group_kb, kscratch, kcount);
    return launch_ok();
}

}  // namespace

int64_t sgemm_3xtf32_scratch_bytes(int64_t pieces) {
    return kSplitKHeaderBytes(pieces) + pieces * (int64_t)(BM * BN * sizeof(float));
}

bool sgemm_3xtf32_supported(const GemmParams& prm) {
    // TMA: 16-byte aligned bases and row pitches; big enough that a 128 x 128 tile is not mostly padding
    const bool aligned = reinterpret_cast<uintptr_t>(prm.A) % 16 == 0 && reinterpret_cast<uintptr_t>(prm.B) % 16 == 0 &&
                         reinterpret_cast<uintptr_t>(prm.C) % 16 == 0;
    const bool pitches = (prm.K % 4 == 0) && (prm.b_kmajor || prm.N % 4 == 0);
    return aligned && pitches && prm.M >= 64 && prm.N >= 64 && prm.K >= 32 && tc::encode_tiled_fn() != nullptr;
}

gpd_status sgemm_3xtf32_launch(const GemmParams& prm, cudaStream_t st) {
    if (prm.b_kmajor) return prm.update ? launch<true, true>(prm, st) : launch<true, false>(prm, st);
    return prm.update ? launch<false, true>(prm, st) : launch<false, false>(prm, st);
}

namespace {
// One warp's lane 0 waits on a barrier nobody arrives at; the wait gives up after `limit` cycles.
__global__ void bounded_wait_selftest_kernel(long long limit) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tc::mbar_wait(&bar, 0, &abort_flag, &g_tf32_status, limit);
    }
}
}  // namespace

gpd_status bounded_wait_selftest_launch(long long limit, cudaStream_t st) {
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(limit);
    return launch_ok();
}

int tf32_device_status_fetch_and_clear() {
    int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_tf32_status, sizeof(int)) != cudaSuccess) return (int)GPD_ERR_CUDA;
    if (v != 0) cudaMemcpyToSymbol(g_tf32_status, &zero, sizeof(int));
    return v;
}

}  // namespace gpd
