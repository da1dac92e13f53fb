// Attention of the kept queries over [prior-scale K/V cache ++ kept tokens' own K/V]
// (no mask), on the sm_100a tensor cores.
//
// One CTA = 256 query rows (two 128-row tiles A and B) of one image and one head, streaming
// over 128-key tiles of K and V:
//   warp 0        TMA producer: Q tiles once, then a ring of K tiles and a ring of V tiles
//   warps 2-3     idle (they fill the producer/issuer warpgroup, which gives up registers)
//   warp 1        tcgen05.mma issuer. Per key tile j:  O_A += P_A V_j ; S_A = Q_A K_{j+1}^T ;
//                 O_B += P_B V_j ; S_B = Q_B K_{j+1}^T.  S and O are fp32 in tensor memory and
//                 O accumulates there across all key tiles.
//   warps 4-7     softmax of tile A, one query row per thread: read the row of S from tensor
//   warps 8-11    memory once, probabilities P = 2^((s - m) * scale) packed to bf16 and stored
//   (tile B)      back into tensor memory over the S columns, from where the next MMA takes them
//                 as its A operand. While one tile's softmax runs, the tensor core works on the
//                 other tile.
// Probabilities are taken against a reference maximum m fixed at the row's first key tile: bf16
// and fp32 share their exponent range, so a reference that is not the running maximum costs no
// precision, and it cancels in the final division by l. Only a score about 2^40 above the
// reference (seen as a huge row sum) raises it, with O and l rescaled in tensor memory; the row
// maximum is therefore not computed on the way. K tiles are K-major operands; V tiles are
// the MN-major B operand, i.e. V is consumed exactly as it lies in the cache ([keys, dh]).
// MMAs issued by one thread execute in issue order, which orders "P_A read by O_A += P_A V" before
// "S_A overwritten by the next Q_A K^T" and "O complete" before the next S of the same tile.
// When the grid's last wave would be less than half full, each of its work items is shared by
// two CTAs that take half of the key tiles each and merge their partial results (see below).
// Every mbarrier wait is bounded.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int BQ = 128;        // query rows per tile (two tiles per CTA)
constexpr int BKV = 128;       // keys per tile
constexpr int kThreads = 384;     // warpgroup 0: producer + MMA issuer (+2 idle warps); 1, 2: softmax of tile A, B
// setmaxnreg.inc waits until the registers are there, and nothing bounds that wait: the split must
// leave slack in the 64 K register file (128 * 64 + 256 * 216 = 63488; a split that used all
// 65536 never got its registers and the kernel hung).
constexpr int kRegsLow = 64, kRegsHigh = 216;
static_assert(128 * kRegsLow + 256 * kRegsHigh <= 65536 - 2048, "keep slack for setmaxnreg.inc");
constexpr int kSlabBytes = 128 * 128;   // [128 rows][64 bf16]
// A row's sum of probabilities over one key tile at or above this (or NaN) means a score about
// 2^40 above the row's reference maximum: the reference is raised and O, l rescaled. Far below
// anything that could overflow fp32 in l or O, far above anything ordinary data reaches.
constexpr float kHugeSum = 1.0995116e12f;   // 2^40

template <int DH>
struct AttnSmem {
    // K_{j+1} is last read by S = Q K_{j+1}^T in step j, V_j by O += P V_j in the same step, one
    // softmax after V_j's own scores, so the two rings have different depths and one release (after
    // the step's last instruction) serves both; head size 128 fills the 227 KB with two Q tiles,
    // three K stages and two V stages.
    static constexpr int kKStages = (DH == 64) ? 4 : 3;
    static constexpr int kVStages = (DH == 64) ? 4 : 2;
    static constexpr int kSlabs = DH / 64;
    static constexpr int kTileBytes = kSlabs * kSlabBytes;      // one 128-row Q, K or V tile
    static constexpr int kQOff = 0;
    static constexpr int kKOff = 2 * kTileBytes;
    static constexpr int kVOff = kKOff + kKStages * kTileBytes;
    static constexpr int kBarOff = kVOff + kVStages * kTileBytes;
    static constexpr int kTotal = kBarOff + 512 + 1024;
};

struct AttnParams {
    const int32_t* cu_keep;
    const int32_t* kv_len;
    __nv_bfloat16* o;
    int B, C, Lmax, n_heads, num_sms;
    int own_keys;          // 1: keys = cache rows followed by this call's k_b rows; 0: cache rows only (cross-attention)
    float scale_log2e;     // (1 / sqrt(dh)) * log2(e)
    // key-split of a last partial wave: per split item two partial results [2][256 rows][DH + 4]
    // fp32 (unnormalised O row, reference maximum, sum) and a ticket counter; part == NULL: no split
    float* part;
    unsigned int* tickets;
    int part_slots;
    unsigned int* status;
};

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}

// ---- two fp32 values per 64-bit register: one instruction does both lanes' arithmetic ----------
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t add_rm_f32x2(uint64_t a, uint64_t b)   // rounds toward -inf
{
    uint64_t r;
    asm("add.rm.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t sub_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// 2^x for two values without the special-function unit, which the softmax would otherwise
// saturate (it evaluates 16 exponentials per clock per SM against 128 multiply-adds). With
// t = x + 1.5 * 2^23 rounded toward -inf, the low bits of t hold j = floor(x) and f = x - j lies in
// [0, 1); 2^f comes from a cubic fitted to 9.2e-5 relative error (far below the bf16 rounding the
// probabilities get next) and j is added to the exponent field as an integer. x is clamped at
// -126 so that the exponent cannot wrap; a masked (-inf) score therefore yields 2^-126, not 0.
__device__ __forceinline__ void exp2_poly_x2(uint64_t x2, float& p0, float& p1)
{
    float x0, x1;
    unpack_f32x2(x2, x0, x1);
    const uint64_t xc = pack_f32x2(fmaxf(x0, -126.f), fmaxf(x1, -126.f));
    const uint64_t magic = pack_f32x2(12582912.f, 12582912.f);
    const uint64_t t = add_rm_f32x2(xc, magic);
    const uint64_t f = sub_f32x2(xc, sub_f32x2(t, magic));
    uint64_t q = fma_f32x2(f, pack_f32x2(0.07711965590715408f, 0.07711965590715408f),
                           pack_f32x2(0.2276432067155838f, 0.2276432067155838f));
    q = fma_f32x2(q, f, pack_f32x2(0.6950892806053162f, 0.6950892806053162f));
    q = fma_f32x2(q, f, pack_f32x2(1.f, 1.f));
    float q0, q1, t0, t1;
    unpack_f32x2(q, q0, q1);
    unpack_f32x2(t, t0, t1);
    p0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(t0) << 23));
    p1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(t1) << 23));
}

template <int DH>
__global__ void __launch_bounds__(kThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                 const __grid_constant__ CUtensorMap tmap_v, const AttnParams p)
{
    using L = AttnSmem<DH>;
    constexpr int kSlabs = L::kSlabs;
    constexpr int kKStages = L::kKStages, kVStages = L::kVStages;
    constexpr int kIssuers = (DH == 128) ? 2 : 1;     // threads that issue tcgen05.mma (see the issuer code below)
    constexpr uint32_t kTmemCols = 512;
    // S tile t (fp32) sits at column 128*t; its first 64 columns are reused for P (bf16 pairs).
    // O tile t (fp32, DH columns) sits at column 256 + 128*t.

    // ---- which (image, 256-row query block, head) is this CTA? ----------------------------
    // Work items are (head, query block), blocks fastest so that CTAs running together share K/V
    // in L2. All items cost the same, so a grid of T items runs in ceil(T / SMs) waves and the last
    // wave may be nearly empty: when it would fill at most half of the SMs, each of its items is
    // run by two CTAs, one per half of the keys. Both leave their unnormalised result (O row,
    // reference maximum, sum) in scratch memory and draw a ticket; the one that draws the second
    // ticket finds the other's result complete, merges the two and writes the output. Nobody
    // waits for anybody.
    int units = 0;
    for (int i = 0; i < p.B; ++i) units += (p.cu_keep[i + 1] - p.cu_keep[i] + 2 * BQ - 1) / (2 * BQ);
    const int items = units * p.n_heads;
    const int rem = items % p.num_sms;
    const bool split = p.part && rem > 0 && 2 * rem <= p.num_sms && rem <= p.part_slots;
    const int whole_items = split ? items - rem : items;
    int item = blockIdx.x, khalf = -1, tail_slot = 0;
    if (item >= whole_items) {
        const int h = item - whole_items;
        item = whole_items + (h >> 1);
        khalf = h & 1;
        tail_slot = h >> 1;
    }
    if (item >= items) return;
    const int head = item / units;
    int slot = item - head * units, b = 0, k_b = 0, q_begin = 0;
    for (b = 0; b < p.B; ++b) {
        const int c0 = p.cu_keep[b];
        k_b = p.cu_keep[b + 1] - c0;
        const int blocks = (k_b + 2 * BQ - 1) / (2 * BQ);
        if (slot < blocks) { q_begin = c0 + slot * 2 * BQ; break; }
        slot -= blocks;
    }
    const int rows_valid = min(2 * BQ, k_b - slot * 2 * BQ);
    const bool tile_b_active = rows_valid > BQ;
    const int n_keys = min(max(p.kv_len[b], 0) + (p.own_keys ? k_b : 0), p.Lmax);
    const int n_tiles_all = (n_keys + BKV - 1) / BKV;
    if (khalf >= 0 && n_tiles_all < 4) {      // too few key tiles to share: the first CTA takes them all
        if (khalf == 1) return;
        khalf = -1;
    }
    if (n_keys == 0) {
        // nothing to attend to (cross-attention with no condition tokens): the output rows are zero
        for (int i = threadIdx.x; i < rows_valid * (DH / 8); i += kThreads) {
            const int r = i / (DH / 8), v = i - r * (DH / 8);
            *(uint4*)(p.o + (long)(q_begin + r) * p.C + head * DH + v * 8) = make_uint4(0, 0, 0, 0);
        }
        return;
    }
    // this CTA's key tiles are jt0 .. jt0 + n_tiles - 1; loops below count j from 0
    int jt0 = 0, n_tiles = n_tiles_all;
    if (khalf == 0) n_tiles = (n_tiles_all + 1) / 2;
    if (khalf == 1) { jt0 = (n_tiles_all + 1) / 2; n_tiles = n_tiles_all - jt0; }

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = (uint64_t*)(smem + L::kBarOff);
    uint64_t* q_full = bars;                          // 1
    uint64_t* k_full = bars + 1;                      // kKStages
    uint64_t* k_empty = k_full + kKStages;            // kKStages
    uint64_t* v_full = k_empty + kKStages;            // kVStages
    uint64_t* s_full = v_full + kVStages;             // 2 (tile A, tile B)
    uint64_t* p_full = s_full + 2;                    // 2, one arrival per softmax warp
    uint64_t* o_done = p_full + 2;                    // 1, one arrival per issuing thread
    uint64_t* turn = o_done + 1;                      // 2 counters (not barriers): turns granted to the issuing thread of tile t
    uint32_t* tmem_slot = (uint32_t*)(turn + 2);
    __shared__ int abort_flag_s;
    __shared__ int ticket_s;
    volatile int* abort_flag = &abort_flag_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        abort_flag_s = 0;
        mbar_init(q_full, 1);
        // a K or V stage is free once the issuing thread of every active query tile has committed
        const int n_issuers = (kIssuers == 2 && tile_b_active) ? 2 : 1;
        for (int s = 0; s < kKStages; ++s) {
            mbar_init(&k_full[s], 1);
            mbar_init(&k_empty[s], n_issuers);
        }
        for (int s = 0; s < kVStages; ++s) mbar_init(&v_full[s], 1);
        for (int t = 0; t < 2; ++t) {
            mbar_init(&s_full[t], 1);
            mbar_init(&p_full[t], 4);
            turn[t] = 0;                              // a plain counter, not a barrier
        }
        mbar_init(o_done, n_issuers);
        fence_barrier_init();
        prefetch_tmap(&tmap_q);
        prefetch_tmap(&tmap_k);
        prefetch_tmap(&tmap_v);
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    uint8_t* q_smem = smem + L::kQOff;

    // The softmax warps hold a whole 128-column row of S in registers; the producer and the MMA
    // issuer need few. Each warpgroup resizes its share of the register file accordingly (the
    // resize must dominate all of the role's code, hence the nesting).
    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsLow));
    if (warp == 0) {
        if (lane == 0) {
            const int q_tiles = tile_b_active ? 2 : 1;
            mbar_arrive_expect_tx(q_full, q_tiles * L::kTileBytes);
            for (int t = 0; t < q_tiles; ++t)
                for (int sl = 0; sl < kSlabs; ++sl)
                    tma_load_2d(q_smem + t * L::kTileBytes + sl * kSlabBytes, &tmap_q, q_full,
                                head * DH + sl * 64, q_begin + t * BQ);
            // order of issue = order in which the slots come free: K_j, V_j, K_{j+1}, ...
            int k_issued = 0, v_issued = 0;
            for (int j = 0; j < n_tiles; ++j) {
                const int ks = j % kKStages, vs = j % kVStages;
                if (j >= kKStages && !mbar_wait(&k_empty[ks], ((j / kKStages) - 1) & 1, abort_flag, p.status)) break;
                uint8_t* k_dst = smem + L::kKOff + ks * L::kTileBytes;
                mbar_arrive_expect_tx(&k_full[ks], L::kTileBytes);
                for (int sl = 0; sl < kSlabs; ++sl)
                    tma_load_3d(k_dst + sl * kSlabBytes, &tmap_k, &k_full[ks], head * DH + sl * 64, (jt0 + j) * BKV, b);
                k_issued = j + 1;
                // The slot of V_j held V_{j-kVStages}, whose last reader is step j-kVStages. That step ends with
                // S = Q K_{j-kVStages+1}^T, and the commit that releases that K tile (k_empty) follows every
                // instruction of the step, O += P V included: it releases the V tile as well. (The K slot is
                // not released again before K_{j-kVStages+1+kKStages} has been loaded, which comes after
                // this wait since kKStages + 1 > kVStages: the phase waited for cannot be overtaken twice.)
                static_assert(kKStages + 1 > kVStages, "the K release that stands for the V release must not be overtaken");
                if (j >= kVStages) {
                    const int kj = j - kVStages + 1;
                    if (!mbar_wait(&k_empty[kj % kKStages], (kj / kKStages) & 1, abort_flag, p.status)) break;
                }
                uint8_t* v_dst = smem + L::kVOff + vs * L::kTileBytes;
                mbar_arrive_expect_tx(&v_full[vs], L::kTileBytes);
                for (int sl = 0; sl < kSlabs; ++sl)
                    tma_load_3d(v_dst + sl * kSlabBytes, &tmap_v, &v_full[vs], head * DH + sl * 64, (jt0 + j) * BKV, b);
                v_issued = j + 1;
            }
            if (*abort_flag) {
                mbar_drain(q_full, 0);
                for (int j = max(0, k_issued - kKStages); j < k_issued; ++j) mbar_drain(&k_full[j % kKStages], (j / kKStages) & 1);
                for (int j = max(0, v_issued - kVStages); j < v_issued; ++j) mbar_drain(&v_full[j % kVStages], (j / kVStages) & 1);
            }
        }
    } else if (warp == 1 || warp == 2) {
        // tcgen05.mma issuers. Per key tile j and query tile t one elected thread issues
        //     O_t += P_t V_j ; S_t = Q_t K_{j+1}^T          (16 instructions at head size 128)
        // Issuing costs a thread about 80 clocks per instruction in this kernel (more than the 64 an
        // instruction executes in) and a satisfied barrier wait 65 to 180.
        if constexpr (kIssuers == 2) {
            // Head size 128: one thread serving both tiles was itself the limit (its waits and loop
            // bookkeeping sat between the two tiles' instruction groups), so each tile has its own thread
            // (warp 1 for tile A, warp 2 for tile B) and all of that happens while the other thread
            // issues. The two pass a token so that the groups still alternate A, B, A, B: left to
            // themselves the tiles drift into phase (both softmaxes at once, then both instruction
            // groups), which is slower than the alternation, where one tile's softmax runs under the
            // other tile's instructions. The token orders instruction issue only; no data depends on it.
            const int t = warp - 1;
            if (lane == 0 && (t == 0 || tile_b_active)) {
                constexpr uint32_t idesc_s = idesc_bf16_f32(BQ, BKV, 0);
                constexpr uint32_t idesc_o = idesc_bf16_f32(BQ, DH, 1);
                // Shared-memory descriptors: (address >> 4) sits in the low 14 bits, so stepping through
                // a tile or to another stage is an integer add.
                constexpr uint32_t kTileStep = L::kTileBytes >> 4;
                const uint64_t q_desc = smem_desc_sw128(smem_u32(q_smem), 16, 1024) + (uint32_t)t * kTileStep;
                const uint64_t k_desc = smem_desc_sw128(smem_u32(smem + L::kKOff), 16, 1024);
                const uint64_t v_desc = smem_desc_sw128(smem_u32(smem + L::kVOff), kSlabBytes, 1024);
                const uint32_t s_tmem = tmem_base + 128u * t, o_tmem = tmem_base + 256u + 128u * t;
                const bool paired = tile_b_active;
                uint32_t turn_par = 0;
                // S_t = Q_t K^T with K in stage ks
                auto issue_s = [&](int ks) {
                    const uint64_t kd = k_desc + (uint32_t)ks * kTileStep;
#pragma unroll
                    for (int kk = 0; kk < DH / 16; ++kk) {
                        constexpr uint32_t kSlabStep = kSlabBytes >> 4;
                        const uint32_t off = (kk >> 2) * kSlabStep + (kk & 3) * 2;    // 32 bytes per 16 k
                        mma_bf16_ss(s_tmem, q_desc + off, kd + off, idesc_s, kk ? 1u : 0u);
                    }
                    mma_commit(&s_full[t]);
                };
                // O_t (+)= P_t V with V in stage vs; P_t sits in the first 64 columns of S_t, two keys per column
                auto issue_pv = [&](int vs, bool first) {
                    const uint64_t vd = v_desc + (uint32_t)vs * kTileStep;
#pragma unroll
                    for (int kk = 0; kk < BKV / 16; ++kk)
                        mma_bf16_ts(o_tmem, s_tmem + kk * 8, vd + (uint32_t)(kk * 128), idesc_o, (first && kk == 0) ? 0u : 1u);
                };
                // the token: wait for this tile's turn, hand the turn to the other tile once this tile's
                // instructions are issued (they execute in the order in which they were issued)
                // (a counter in shared memory polled with plain loads: the waiting thread has nothing else to
                // do, and a load comes back several times faster than a suspended barrier wait wakes up)
                volatile uint32_t* turn_ctr = (volatile uint32_t*)turn;      // [2], zeroed with the barriers
                auto take_turn = [&]() {
                    if (!paired) return true;
                    ++turn_par;                                   // number of the turn this thread waits for
                    if (turn_ctr[t * 2] >= turn_par) return true;
                    const unsigned long long t0 = global_ns();
                    uint32_t spins = 0;
                    while (turn_ctr[t * 2] < turn_par) {
                        if ((++spins & 255u) == 0) {
                            if (*abort_flag) return false;
                            unsigned long long limit = *(volatile const unsigned long long*)(p.status + NOVA_WAIT_LIMIT_WORD);
                            if (limit == 0) limit = kWaitLimitNs;
                            if (global_ns() - t0 > limit) {
                                *abort_flag = 1;
                                atomicOr(p.status, NOVA_DEV_TIMEOUT);
                                return false;
                            }
                        }
                    }
                    return true;
                };
                uint32_t passed = 0;
                auto pass_turn = [&]() {
                    if (!paired) return;
                    turn_ctr[(t ^ 1) * 2] = ++passed;      // no fence: the token orders issue in time, no data hangs on it
                };
                bool ok = mbar_wait(q_full, 0, abort_flag, p.status);
                if (ok) ok = mbar_wait(&k_full[0], 0, abort_flag, p.status);
                if (ok && t == 1) ok = take_turn();          // tile A goes first
                if (ok) {
                    tc_fence_after();
                    issue_s(0);
                    mma_commit(&k_empty[0]);
                    pass_turn();
                }
                // ring positions and phase parities, stepped without divisions
                int vs = 0, ks_next = (kKStages > 1) ? 1 : 0;
                uint32_t v_par = 0, k_par_next = (kKStages > 1) ? 0u : 1u;
                for (int j = 0; j < n_tiles && ok; ++j) {
                    const bool more = j + 1 < n_tiles;
                    // V_j and K_{j+1} have usually landed long ago; P is what a step waits for
                    ok = mbar_wait(&v_full[vs], v_par, abort_flag, p.status);
                    if (ok && more) ok = mbar_wait(&k_full[ks_next], k_par_next, abort_flag, p.status);
                    if (ok && !mbar_test_wait(&p_full[t], j & 1)) {
                        // polled without suspending: this thread has nothing else to do
                        const unsigned long long t0 = global_ns();
                        uint32_t spins = 0;
                        while (!mbar_test_wait(&p_full[t], j & 1)) {
                            if ((++spins & 255u) == 0) {
                                if (*abort_flag) { ok = false; break; }
                                unsigned long long limit = *(volatile const unsigned long long*)(p.status + NOVA_WAIT_LIMIT_WORD);
                                if (limit == 0) limit = kWaitLimitNs;
                                if (global_ns() - t0 > limit) {
                                    *abort_flag = 1;
                                    atomicOr(p.status, NOVA_DEV_TIMEOUT);
                                    ok = false;
                                    break;
                                }
                            }
                        }
                    }
                    if (ok) ok = take_turn();
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(vs, j == 0);
                    if (more) {
                        issue_s(ks_next);
                        mma_commit(&k_empty[ks_next]);              // this tile no longer reads K_{j+1}, nor V_j
                    }
                    pass_turn();
                    if (++vs == kVStages) { vs = 0; v_par ^= 1u; }
                    if (++ks_next == kKStages) { ks_next = 0; k_par_next ^= 1u; }
                }
                if (ok) mma_commit(o_done);
            }
        } else if (warp == 1) {
            // Head size 64: the groups are short, the token costs more than it saves, and one thread
            // serves both tiles in the fixed order A, B.
            if (lane == 0) {
                constexpr uint32_t idesc_s = idesc_bf16_f32(BQ, BKV, 0);
                constexpr uint32_t idesc_o = idesc_bf16_f32(BQ, DH, 1);
                // Shared-memory descriptors: (address >> 4) sits in the low 14 bits, so stepping through
                // a tile or to another stage is an integer add.
                constexpr uint32_t kTileStep = L::kTileBytes >> 4;
                const uint64_t q_desc = smem_desc_sw128(smem_u32(q_smem), 16, 1024);
                const uint64_t k_desc = smem_desc_sw128(smem_u32(smem + L::kKOff), 16, 1024);
                const uint64_t v_desc = smem_desc_sw128(smem_u32(smem + L::kVOff), kSlabBytes, 1024);
                const int n_q = tile_b_active ? 2 : 1;
                // S_t = Q_t K^T with K in stage ks
                auto issue_s = [&](int t, int ks) {
                    const uint64_t qd = q_desc + (uint32_t)t * kTileStep;
                    const uint64_t kd = k_desc + (uint32_t)ks * kTileStep;
#pragma unroll
                    for (int kk = 0; kk < DH / 16; ++kk) {
                        constexpr uint32_t kSlabStep = kSlabBytes >> 4;
                        const uint32_t off = (kk >> 2) * kSlabStep + (kk & 3) * 2;    // 32 bytes per 16 k
                        mma_bf16_ss(tmem_base + 128u * t, qd + off, kd + off, idesc_s, kk ? 1u : 0u);
                    }
                    mma_commit(&s_full[t]);
                };
                // O_t (+)= P_t V with V in stage vs; P_t sits in the first 64 columns of S_t, two keys per column
                auto issue_pv = [&](int t, int vs, bool first) {
                    const uint64_t vd = v_desc + (uint32_t)vs * kTileStep;
#pragma unroll
                    for (int kk = 0; kk < BKV / 16; ++kk)
                        mma_bf16_ts(tmem_base + 256u + 128u * t, tmem_base + 128u * t + kk * 8, vd + (uint32_t)(kk * 128),
                                    idesc_o, (first && kk == 0) ? 0u : 1u);
                };
                bool ok = mbar_wait(q_full, 0, abort_flag, p.status);
                if (ok) ok = mbar_wait(&k_full[0], 0, abort_flag, p.status);
                if (ok) {
                    tc_fence_after();
                    for (int t = 0; t < n_q; ++t) issue_s(t, 0);
                    mma_commit(&k_empty[0]);
                }
                // ring positions and phase parities, stepped without divisions
                int vs = 0, ks_next = (kKStages > 1) ? 1 : 0;
                uint32_t v_par = 0, k_par_next = (kKStages > 1) ? 0u : 1u;
                for (int j = 0; j < n_tiles && ok; ++j) {
                    const bool more = j + 1 < n_tiles;
                    // V_j and K_{j+1} have usually landed long ago; P is what a step waits for
                    ok = mbar_wait(&v_full[vs], v_par, abort_flag, p.status);
                    if (ok && more) ok = mbar_wait(&k_full[ks_next], k_par_next, abort_flag, p.status);
                    for (int t = 0; t < n_q && ok; ++t) {
                        ok = mbar_wait(&p_full[t], j & 1, abort_flag, p.status);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(t, vs, j == 0);
                        if (more) {
                            issue_s(t, ks_next);
                            if (t == n_q - 1) mma_commit(&k_empty[ks_next]);        // K_{j+1} and V_j have no reader left
                        }
                    }
                    if (++vs == kVStages) { vs = 0; v_par ^= 1u; }
                    if (++ks_next == kKStages) { ks_next = 0; k_par_next ^= 1u; }
                }
                if (ok) mma_commit(o_done);
            }
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsHigh));
        const int t = (warp >= 8) ? 1 : 0;            // which query tile this warpgroup owns
        if (t == 0 || tile_b_active) {
            const int q = warp & 3;
            const int row = q * 32 + lane;               // row within the tile = TMEM lane
            const uint32_t lane_off = (uint32_t)(q * 32) << 16;
            const uint32_t s_addr = tmem_base + lane_off + 128u * t;
            const uint32_t o_addr = tmem_base + lane_off + 256u + 128u * t;
            const float c = p.scale_log2e;
            // Polynomial share of the exponentials (pairs out of every four pairs of scores). The
            // special-function unit delivers one exponential per 8 clocks and scheduler; the polynomial
            // costs a scheduler about as much in issue slots, so it does not replace that unit, it only
            // works beside it: a quarter of the scores on the polynomial measured best at both head sizes
            // (6.9 clocks per score and scheduler against 7.5 at a half and 8.2 with none).
            constexpr int kPolyPairs = 1;
            // The reference maximum starts at a finite floor, not -inf: (-inf) - (-inf) must not appear.
            float m_ref = -1e30f, l_run = 0.f;
            bool ok = true;
            for (int j = 0; j < n_tiles && ok; ++j) {
                ok = mbar_wait_warp(&s_full[t], j & 1, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
                const int cols_valid = n_keys - (jt0 + j) * BKV;      // >= 1; < BKV only on a ragged last tile
                // the whole row of S (128 scores) into registers with one round trip to tensor memory
                uint32_t sv[128];
#pragma unroll
                for (int cch = 0; cch < 4; ++cch)
                    tmem_ld32(s_addr + cch * 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[cch * 32]));
                tmem_ld_wait();
                if (cols_valid < BKV) {
#pragma unroll
                    for (int i = 0; i < 128; ++i)
                        if (i >= cols_valid) sv[i] = 0xff800000u;   // -inf: key past the end
                }
                auto row_max = [&]() {
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int i = 0; i < 128; i += 8) {
#pragma unroll
                        for (int a = 0; a < 4; ++a)
                            mx4[a] = fmax3(mx4[a], __uint_as_float(sv[i + 2 * a]), __uint_as_float(sv[i + 2 * a + 1]));
                    }
                    return fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                };
                if (j == 0) m_ref = fmaxf(m_ref, row_max());      // the row's reference: its maximum over the first key tile
                // p = 2^(s*c - m*c), 32 scores at a time: 16 registers of bf16 pairs each, written over the
                // first columns of S as they are ready. Returns the sum of the 128 probabilities.
                auto exponentials = [&](bool store) {
                    const uint64_t c2 = pack_f32x2(c, c);
                    const uint64_t nm2 = pack_f32x2(-m_ref * c, -m_ref * c);
                    uint64_t lsum_a = pack_f32x2(0.f, 0.f), lsum_b = lsum_a;
#pragma unroll
                    for (int cch = 0; cch < 4; ++cch) {
                        uint32_t pk[16];
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const int i = cch * 32 + 8 * g + 2 * q;
                                const uint64_t y = fma_f32x2(pack_f32x2(__uint_as_float(sv[i]), __uint_as_float(sv[i + 1])), c2, nm2);
                                float p0, p1;
                                if (q < kPolyPairs) {
                                    exp2_poly_x2(y, p0, p1);
                                } else {
                                    float y0, y1;
                                    unpack_f32x2(y, y0, y1);
                                    p0 = ex2(y0);
                                    p1 = ex2(y1);
                                }
                                if (q & 1) lsum_b = add_f32x2(lsum_b, pack_f32x2(p0, p1));
                                else lsum_a = add_f32x2(lsum_a, pack_f32x2(p0, p1));
                                pk[4 * g + q] = pack_bf16(p0, p1);
                            }
                        }
                        if (store) tmem_st16(s_addr + cch * 16, pk);
                    }
                    float s0, s1, s2, s3;
                    unpack_f32x2(lsum_a, s0, s1);
                    unpack_f32x2(lsum_b, s2, s3);
                    return (s0 + s2) + (s1 + s3);
                };
                float lsum = exponentials(true);
                if (j > 0 && __any_sync(0xffffffffu, !(lsum < kHugeSum))) {
                    // a score far above the reference: raise it, rescale what has been accumulated
                    // (the tile's previous O += P V is complete: its S could not have been written
                    // otherwise) and take the tile's probabilities again
                    const float m_new = fmaxf(m_ref, row_max());
                    const float alpha = ex2((m_ref - m_new) * c);
                    tmem_st_wait();
#pragma unroll
                    for (int cch = 0; cch < DH / 32; ++cch) {
                        uint32_t ov[32];
                        tmem_ld32(o_addr + cch * 32, ov);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
                        tmem_st32(o_addr + cch * 32, ov);
                    }
                    l_run *= alpha;
                    m_ref = m_new;
                    lsum = exponentials(true);
                }
                l_run += lsum;
                tmem_st_wait();
                if ((t == 0 || kIssuers == 2) && cols_valid < BKV) {
                    // ragged last tile: rows of V past the last key may hold anything (even NaN);
                    // zero them so that 0 * garbage cannot poison the accumulator. With one issuing
                    // thread tile A's O += P V is issued before tile B's, so tile A's softmax warps do it
                    // for both; with a thread per tile each tile's warps do it before their own hand-over
                    // (zeros written over zeros are harmless)
                    const int s = j % kVStages;
                    ok = mbar_wait_warp(&v_full[s], (j / kVStages) & 1, abort_flag, p.status);
                    if (!ok) break;
                    if (row >= cols_valid) {
                        uint8_t* v_row = smem + L::kVOff + s * L::kTileBytes + row * 128;
#pragma unroll
                        for (int sl = 0; sl < kSlabs; ++sl)
#pragma unroll
                            for (int g = 0; g < 8; ++g) *(uint4*)(v_row + sl * kSlabBytes + g * 16) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async_smem();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_full[t]);
            }
            if (ok) ok = mbar_wait_warp(o_done, 0, abort_flag, p.status);
            const int grow = t * BQ + row;
            __nv_bfloat16* dst_row = p.o + (long)(q_begin + grow) * p.C + head * DH;
            if (ok && khalf < 0) {
                tc_fence_after();
                const float inv = 1.f / l_run;
#pragma unroll
                for (int cch = 0; cch < DH / 32; ++cch) {
                    uint32_t ov[32];
                    tmem_ld32(o_addr + cch * 32, ov);
                    tmem_ld_wait();
                    if (grow < rows_valid) {
                        uint4* dst = (uint4*)(dst_row + cch * 32);
#pragma unroll
                        for (int g = 0; g < 4; ++g)
                            dst[g] = make_uint4(
                                pack_bf16(__uint_as_float(ov[g * 8]) * inv, __uint_as_float(ov[g * 8 + 1]) * inv),
                                pack_bf16(__uint_as_float(ov[g * 8 + 2]) * inv, __uint_as_float(ov[g * 8 + 3]) * inv),
                                pack_bf16(__uint_as_float(ov[g * 8 + 4]) * inv, __uint_as_float(ov[g * 8 + 5]) * inv),
                                pack_bf16(__uint_as_float(ov[g * 8 + 6]) * inv, __uint_as_float(ov[g * 8 + 7]) * inv));
                    }
                }
            } else if (khalf >= 0) {
                // ---- half of the keys: publish the partial result, then merge if the other is there
                // (all softmax threads of the CTA take part, also after a failed wait, so that the
                // named barrier below is complete; a failed CTA publishes nothing useful and the
                // status word says so)
                constexpr int kStride = DH + 4;
                float* mine = p.part + ((size_t)(tail_slot * 2 + khalf) * (2 * BQ) + grow) * kStride;
                const float* other = p.part + ((size_t)(tail_slot * 2 + (khalf ^ 1)) * (2 * BQ) + grow) * kStride;
                if (ok) {
                    tc_fence_after();
#pragma unroll
                    for (int cch = 0; cch < DH / 32; ++cch) {
                        uint32_t ov[32];
                        tmem_ld32(o_addr + cch * 32, ov);
                        tmem_ld_wait();
#pragma unroll
                        for (int g = 0; g < 8; ++g)
                            *(uint4*)(mine + cch * 32 + g * 4) = make_uint4(ov[g * 4], ov[g * 4 + 1], ov[g * 4 + 2], ov[g * 4 + 3]);
                    }
                    mine[DH] = m_ref;
                    mine[DH + 1] = l_run;
                }
                __threadfence();
                const int n_soft = tile_b_active ? 256 : 128;
                asm volatile("bar.sync 1, %0;" ::"r"(n_soft) : "memory");
                if (threadIdx.x == 128) {
                    const unsigned int ticket = atomicAdd(&p.tickets[tail_slot], 1u);
                    if (ticket == 1u) p.tickets[tail_slot] = 0;          // ready for the next launch
                    ticket_s = (int)ticket;
                }
                asm volatile("bar.sync 1, %0;" ::"r"(n_soft) : "memory");
                if (ok && ticket_s == 1) {
                    // the other CTA fenced its partial result before it drew ticket 0
                    // The merge is written in terms of (half 0, half 1), not (mine, other), with every
                    // rounding spelled out: either CTA may be the one that merges, and the output must
                    // not depend on which.
                    const float m_o = __ldcg(other + DH), l_o = __ldcg(other + DH + 1);
                    const float m_new = fmaxf(m_ref, m_o);
                    const float a_me = ex2((m_ref - m_new) * c), a_o = ex2((m_o - m_new) * c);
                    const bool first = (khalf == 0);
                    const float a0 = first ? a_me : a_o, a1 = first ? a_o : a_me;
                    const float l0 = first ? l_run : l_o, l1 = first ? l_o : l_run;
                    const float inv = 1.f / __fmaf_rn(l0, a0, __fmul_rn(l1, a1));
                    const float w0 = a0 * inv, w1 = a1 * inv;
                    const float w_me = first ? w0 : w1, w_o = first ? w1 : w0;
                    auto mix = [&](uint32_t mine_bits, float theirs) {
                        const float me = __uint_as_float(mine_bits);
                        // half 0's term is the multiply-add operand, half 1's the rounded product
                        return first ? __fmaf_rn(me, w_me, __fmul_rn(theirs, w_o))
                                     : __fmaf_rn(theirs, w_o, __fmul_rn(me, w_me));
                    };
#pragma unroll
                    for (int cch = 0; cch < DH / 32; ++cch) {
                        uint32_t ov[32];
                        tmem_ld32(o_addr + cch * 32, ov);
                        tmem_ld_wait();
                        if (grow < rows_valid) {
                            uint4* dst = (uint4*)(dst_row + cch * 32);
#pragma unroll
                            for (int g = 0; g < 4; ++g) {
                                const float4 o0 = __ldcg((const float4*)(other + cch * 32 + g * 8));
                                const float4 o1 = __ldcg((const float4*)(other + cch * 32 + g * 8 + 4));
                                dst[g] = make_uint4(
                                    pack_bf16(mix(ov[g * 8], o0.x), mix(ov[g * 8 + 1], o0.y)),
                                    pack_bf16(mix(ov[g * 8 + 2], o0.z), mix(ov[g * 8 + 3], o0.w)),
                                    pack_bf16(mix(ov[g * 8 + 4], o1.x), mix(ov[g * 8 + 5], o1.y)),
                                    pack_bf16(mix(ov[g * 8 + 6], o1.z), mix(ov[g * 8 + 7], o1.w)));
                            }
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

template <int DH>
nova_status launch(nova_ctx* ctx, const nova_attn_args& a, cudaStream_t st)
{
    using L = AttnSmem<DH>;
    CUtensorMap tq, tk, tv;
    const uint64_t dq[2] = {(uint64_t)a.C, (uint64_t)a.M}, sq[1] = {(uint64_t)a.C * 2};
    const uint64_t dk[3] = {(uint64_t)a.C, (uint64_t)a.Lmax, (uint64_t)a.B};
    const uint64_t sk[2] = {(uint64_t)a.C * 2, (uint64_t)a.Lmax * a.C * 2};
    if (!make_tmap_bf16(ctx, &tq, a.q, 2, dq, sq, BQ) || !make_tmap_bf16(ctx, &tk, a.k_cache, 3, dk, sk, BKV) ||
        !make_tmap_bf16(ctx, &tv, a.v_cache, 3, dk, sk, BKV))
        return nova_fail(ctx, NOVA_ERR_CUDA, "attention: cuTensorMapEncodeTiled failed");
    auto kern = attention_kernel<DH>;
    if (!ctx->attr_attn) {   // both head sizes opt in once per context
        NOVA_CUDA_CHECK(ctx, cudaFuncSetAttribute(attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<64>::kTotal));
        NOVA_CUDA_CHECK(ctx, cudaFuncSetAttribute(attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<128>::kTotal));
        ctx->attr_attn = true;
    }
    AttnParams p;
    p.cu_keep = a.cu_keep; p.kv_len = a.kv_len; p.o = a.o; p.B = a.B; p.C = a.C; p.Lmax = a.Lmax;
    p.scale_log2e = (float)((1.0 / sqrt((double)DH)) * 1.4426950408889634);
    p.status = ctx->dev_status;
    p.n_heads = a.n_heads; p.num_sms = ctx->num_sms;
    p.own_keys = a.cache_only ? 0 : 1;
    // scratch for a key-split last wave: [slots][2][256][DH + 4] fp32; tickets live in the context's
    // status allocation (zero at creation, reset by the CTA that draws the second ticket)
    const size_t slot_bytes = (size_t)2 * 2 * BQ * (DH + 4) * sizeof(float);
    p.part = (float*)a.scratch;
    p.part_slots = a.scratch ? (int)min((size_t)NOVA_ATTN_TICKETS, a.scratch_bytes / slot_bytes) : 0;
    p.tickets = ctx->dev_status + NOVA_ATTN_TICKET_WORD0;
    // upper bound of the work items (the kept counts per image live on the device) plus the CTAs a
    // split last wave adds; CTAs past the end return at once
    dim3 grid(((a.M + 2 * BQ - 1) / (2 * BQ) + a.B) * a.n_heads + ctx->num_sms / 2);
    {
        nova_launch_scope scope(ctx, NOVA_K_ATTENTION, st);
        kern<<<grid, kThreads, L::kTotal, st>>>(tq, tk, tv, p);
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

}  // namespace

nova_status nova_launch_attention(nova_ctx* ctx, const nova_attn_args& a, cudaStream_t st)
{
    if (a.M <= 0) return NOVA_OK;
    const int dh = a.C / a.n_heads;
    if (dh == 64) return launch<64>(ctx, a, st);
    if (dh == 128) return launch<128>(ctx, a, st);
    return nova_fail(ctx, NOVA_ERR_SHAPE, "attention: head dimension must be 64 or 128");
}
