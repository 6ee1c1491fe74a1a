// k2d_kernels.cuh -- device code of the batched 2D rigid-body environment step (sm_100a).
//
// One group of G lanes (G = 16: two scenes per warp; 32: one warp per scene; 8: four scenes per warp)
// owns one scene.  A group takes work items (a run of consecutive steps of one env) from a ticket queue;
// for an item it loads the scene's state from memory once, keeps it in shared memory (bodies, joint rows,
// world-frame geometry) and in registers (the contact pair record of every lane) across the item's steps,
// and writes it back once.  Within a step the lanes of the group work on bodies, polygon vertices, shape
// pairs (bounding-box test, narrowphase), contact pair records (one per lane) and joints (one per lane).
//
// Arithmetic contract: every +,-,*,/,sqrt is an individually rounded IEEE binary32 operation
// (the file is compiled with --fmad=false --prec-div=true --prec-sqrt=true --ftz=false), a fused
// multiply-add appears only where the code says __fmaf_rn, and min/max are comparisons.  The
// sequential-impulse solver keeps the canonical constraint order (joints, then contacts by pair
// index) by "level scheduling": a row's level is one more than the highest level of an earlier
// row that shares a movable body with it, rows of one level touch disjoint movable bodies and
// run on different lanes at once, and levels run in order -- every body sees exactly the
// sequence of updates a one-row-at-a-time sweep would give it, so results are bit-identical to
// that sweep.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace k2d {

// The step kernel runs in blocks of kSmallBlock threads (several blocks per SM, for launches that do not fill the device) or in
// one block per SM of up to kLargeBlock threads (see step_block_threads), in which the warps that share a scheduler step in
// lockstep.  kStepRegisters bounds the kernel's registers: 65536 / 96 = 682 threads per SM.
constexpr int kSmallBlock = 128, kSmallBlocksPerSM = 5, kLargeBlock = 640;
constexpr size_t kMaxBlockSmem = 227 * 1024;
constexpr int kObsThreads = 128;   // observation kernel: one half-warp per env, eight envs per block
constexpr int kMaxActions = 16;
enum { Q_TICKET = 0, Q_LEFT = 1, Q_ERROR = 2 };
constexpr unsigned kWaitLimit = 1u << 24;   // default number of polls (about 100 ns apart) before a wait for another group's chunk gives up
constexpr int kRecWords = 24;   // contact pair record
constexpr int kWarmWords = 5;   // pair index + 4 accumulated impulses
constexpr int kStageWords = 9;  // packed pair word, normal, two contact points with penetration
constexpr int kJointWords = 24; // joint row kept in shared memory: six 16-byte groups
constexpr int kJointLevelWords = 12;  // joint record of a level

// ---------------------------------------------------------------- size classes and layouts
template <int P_, int C_, int J_, int T_>
struct SizeClass {
    static constexpr int P = P_, C = C_, N = P_ + C_, J = J_, T = T_;
    static constexpr int NPP = P * (P - 1) / 2, NPC = P * C, NCC = C * (C - 1) / 2;
    static constexpr int NPAIRS = NPP + NPC + NCC, NSLOTS = 2 * NPP + NPC + NCC;
    static constexpr int MASKW = (NPAIRS + 31) / 32;
    static constexpr int P4 = 4 * P;
    // level record (32-bit words)
    static constexpr int LV_X = 0, LV_Y = N, LV_TH = 2 * N, LV_VX = 3 * N, LV_VY = 4 * N, LV_W = 5 * N;
    static constexpr int LV_IM = 6 * N, LV_II = 7 * N, LV_FR = 8 * N, LV_RE = 9 * N, LV_FLAGS = 10 * N, LV_DENS = 11 * N;
    static constexpr int LV_RAD = 12 * N;
    static constexpr int LV_PVX = LV_RAD + C, LV_PVY = LV_PVX + P4, LV_PNX = LV_PVY + P4, LV_PNY = LV_PNX + P4, LV_ELEN = LV_PNY + P4;
    // J x 12: packed, anchor a xy, anchor b xy, speed, power, fixed angle, lower limit, upper limit, kind (1 fixed, 2 limited), pad
    static constexpr int LV_JOINT = LV_ELEN + P4;
    static constexpr int LV_THR = LV_JOINT + kJointLevelWords * J;      // T x 8: packed, pos xy, dir xy, power, pad, pad
    static constexpr int LV_MASK = LV_THR + 8 * T;
    static constexpr int LV_GB = LV_MASK + MASKW;        // first green shape | first blue shape << 8 | both exist << 16
    static constexpr int LV_WORDS = (LV_GB + 1 + 3) / 4 * 4;
    // state record: bodies (same order as shared memory), joint impulses, meta, warm list
    static constexpr int ST_BODY = 0, ST_JACC = 6 * N, ST_META = ST_JACC + 3 * J, ST_WARM = ST_META + 8;
    static constexpr int ST_WORDS = (ST_WARM + kWarmWords * NPAIRS + 3) / 4 * 4;
    // A scene with more touching pairs than lanes takes the step's contact solve through global
    // scratch: one memory record and one warm entry per pair.
    static constexpr int SCRATCH_WORDS = NPAIRS * (kRecWords + kWarmWords);
    static constexpr int SCRATCH_WARM = NPAIRS * kRecWords;
    // shared memory region of one scene (words)
    // per body 16-byte groups (x, y, angle, -) and (vx, vy, angular velocity, -), then per-body arrays
    static constexpr int BPOS = 0, BVEL = 4 * N;
    static constexpr int BIM = 8 * N, BII = 9 * N, BFR = 10 * N, BRE = 11 * N, BC = 12 * N, BS = 13 * N, BFL = 14 * N;
    static constexpr int RAD = 15 * N;
    static constexpr int WVX = (RAD + C + 3) / 4 * 4, WVY = WVX + P4, WNX = WVY + P4, WNY = WNX + P4, WOFF = WNY + P4;
    static constexpr int BOX = (WOFF + P4 + 3) / 4 * 4;  // N x (min x, min y, max x, max y), 16-byte aligned
    static constexpr int MASK = BOX + 4 * N;
    static constexpr int ACT = MASK + MASKW;
    static constexpr int META = ACT + kMaxActions;       // step_count, episode_count, level_id, status, warm entries
    static constexpr int JROW = (META + 8 + 3) / 4 * 4;  // J rows of kJointWords, 16-byte aligned
    static constexpr int LVC = JROW + kJointWords * J;   // copy of the level record's edge lengths, joint and thruster records
    static constexpr int LVC_WORDS = LV_MASK - LV_ELEN;
    static constexpr int SURV = LVC + LVC_WORDS;         // bytes: pairs that passed the box test
    static constexpr int WIDX = SURV + ((NPAIRS + 3) / 4 > N ? (NPAIRS + 3) / 4 : N); // bytes: pair -> record index of the previous step (the survivor area is reused as N words)
    // then, per lane of the group (field-major, G words per field):
    //   STG  kStageWords fields: manifolds on their way to the owning lane; afterwards the second manifold's constants
    //   ACC2 2 fields: accumulated impulses of the second manifold
    // (the positional corrections of a lane's record, 2 x G words, reuse the world-frame vertex arrays after the narrowphase)
    // then kRecWords fields of G / 2 words: second records of the lower half of the lanes
    static constexpr int STG = WIDX + (NPAIRS + 3) / 4;
    static constexpr int LANE_FIELDS = kStageWords + 2;
    static constexpr int PTAB_WORDS = ((NPAIRS + 1) / 2 + 3) / 4 * 4;  // block-shared pair table, 16 bits per pair
};
// memory form of a contact pair record (the overflow path keeps records in global scratch)
enum { R_AB = 0, R_NX, R_NY, R_MU, R_M0 = 4 };
enum { M_RNA = 0, M_RNB, M_RTA, M_RTB, M_MASSN, M_MASST, M_TARGET, M_CORR, M_ACCN, M_ACCT, M_WORDS };
static_assert(R_M0 + 2 * M_WORDS == kRecWords, "record size");
// staged manifold fields
enum { S_AB = 0, S_NX, S_NY, S_PX0, S_PY0, S_PEN0, S_PX1, S_PY1, S_PEN1 };
static_assert(S_PEN1 + 1 == kStageWords, "stage size");
// second-manifold constants reuse the stage fields of the same lane
enum { M2_RNA = 0, M2_RNB, M2_RTA, M2_RTB, M2_MASSN, M2_MASST, M2_TARGET };
// per-lane fields after the stage fields
enum { LF_ACC2N = kStageWords, LF_ACC2T, LF_COUNT };
// The lower half of the lanes can hold a second record each (pair number G + lane of a crowded scene),
// in memory form: kRecWords fields of G / 2 words after the per-lane fields.  Stage field f of such a
// record waits in record field ovs(f), clear of the accumulated impulses.
__host__ __device__ constexpr int ovs(int f) { return f < 3 ? f : f + 1; }
constexpr int OV_ACC0N = R_M0 + M_ACCN, OV_ACC0T = R_M0 + M_ACCT, OV_ACC1N = R_M0 + M_WORDS + M_ACCN, OV_ACC1T = R_M0 + M_WORDS + M_ACCT;
// joint row fields
enum { JR_RAX = 0, JR_RAY, JR_RBX, JR_RBY, JR_I11, JR_I12, JR_I22, JR_PAD0, JR_BX, JR_BY, JR_CX, JR_CY, JR_MA, JR_MB, JR_IA, JR_IB,
       JR_ACCX, JR_ACCY, JR_PAD1, JR_PAD2,
       JR_ANG, JR_KR, JR_BIASR, JR_ACCR };   // angular row: kind (0 none, 1 fixed, 2 beyond the upper limit, 3 beyond the lower), 1 / (1/I_a + 1/I_b), gamma x error, accumulated
static_assert(JR_ACCR + 1 == kJointWords, "joint row size");
enum { META_STEP = 0, META_EPISODE, META_LEVEL, META_STATUS, META_NWARM, META_GB, META_D0 };   // the last two: dense reward's shapes and distance before the step

// shared-memory word of word i of a state record's body block (x[N], y[N], angle[N], vx[N], vy[N], w[N])
template <class SC>
__device__ __forceinline__ int body_word(int i) {
    const int f = i / SC::N, b = i - f * SC::N;
    return (f < 3 ? SC::BPOS + f : SC::BVEL + f - 3) + 4 * b;
}
// shared-memory words per scene: padded so that the groups of one warp start in different banks
template <class SC, int G>
__host__ __device__ constexpr int region_words() {
    constexpr int raw = SC::STG + SC::LANE_FIELDS * G + kRecWords * (G / 2);
    return G < 32 ? (raw - G + 31) / 32 * 32 + G : (raw + 3) / 4 * 4;
}

// shared memory of a step-kernel block of `threads` threads, and the threads of the one-block-per-SM form: the largest
// multiple of 128 up to kLargeBlock whose scenes fit into an SM's shared memory
template <class SC, int G>
__host__ __device__ constexpr size_t step_block_smem(int threads) {
    return sizeof(uint32_t) * (size_t)(SC::PTAB_WORDS + (threads / G) * region_words<SC, G>());
}
template <class SC, int G>
__host__ __device__ constexpr int step_block_threads() {
    int t = kLargeBlock;
    while (t > kSmallBlock && step_block_smem<SC, G>(t) + 1024 > kMaxBlockSmem) t -= 128;
    return t;
}

// body flag word
constexpr uint32_t F_ACTIVE = 1u, F_DYNAMIC = 2u;
__host__ __device__ inline uint32_t flag_role(uint32_t f) { return (f >> 2) & 3u; }
__host__ __device__ inline uint32_t flag_nverts(uint32_t f) { return (f >> 4) & 7u; }
// joint packed word: a | b<<8 | binding<<16 | on<<24 | level<<25 | active<<28 | a movable<<29 | b movable<<30 | fixed or limited<<31
// thruster packed word: shape | binding<<8 | on<<16 | level<<17 | active<<20
// record AB word: a | b<<5 | amask<<10 | pair<<12 | level<<19 | dynA<<26 | dynB<<27

struct StepParams {
    uint32_t *state;
    const uint32_t *levels;
    const float *actions;
    float *reward;
    uint8_t *done;
    unsigned long long *counters;
    unsigned int *queue;       // work queue words: next ticket, groups that have left, error flag
    unsigned int *chunks_done; // per env: chunks of this launch already stepped (0 again when the launch is over)
    const int *order;          // the envs in the order the launch hands them out (null: by index)
    uint32_t *scratch;
    float *trace;
    float *obs;               // k2d_step_obs: the symbolic observation after the call's last step, [n_envs][obs_floats]; else null
    int n_polygons, n_circles, n_joints, n_thrusters;      // the caller's scene dimensions (observation layout)
    int n_envs, n_steps, n_actions, n_levels;
    int chunk_steps, n_chunks;   // a launch is cut into n_chunks pieces of chunk_steps steps; work items are (chunk, env)
    unsigned wait_limit;         // polls before a wait for another group's chunk gives up
    int n_slots;                 // scratch slots the caller's buffer holds (one per resident scene group)
    int n_batches;               // batched contact solve: number of batches the manifold slots are cut into (0: the sequential sweep)
    int solver_iters, warm_start, auto_reset, max_episode_steps;
    int discrete;             // actions are int32 codes (multi-discrete action space) instead of floats
    int frame_skip;           // engine steps each action row is held for
    float dense_kappa;        // coefficient of the dense reward (0 = off)
    float dt, gdt, contact_alpha, contact_beta, slop, rest_thr, face_tol, joint_alpha, joint_beta, joint_gamma, motor_rho, aabb_margin;
    unsigned long long seed;
    long long env_offset;
};

// ---------------------------------------------------------------- index checks of the checked build
// With -DK2D_CHECKED every index that is unpacked from a packed word or read from a table (bodies, pairs, memory records,
// level ids, warm entries, solver levels, scratch slots, counts) is compared with its limit before it is used; a violation
// sets a bit in k2d_check_bits, which k2d_status reports, and the access goes to index 0 instead.  Nothing traps.  In the
// ordinary build the checks compile to nothing.
enum { CK_BODY = 0, CK_PAIR, CK_RECORD, CK_LEVEL_ID, CK_COUNT, CK_SLOT, CK_WARM, CK_SOLVER_LEVEL, CK_STAGE, CK_OBS };
#ifdef K2D_CHECKED
__device__ unsigned int k2d_check_bits;
template <int CODE>
__device__ __forceinline__ int ck_idx(int v, int limit) {
    if ((unsigned)v >= (unsigned)limit) { atomicOr(&k2d_check_bits, 1u << CODE); return 0; }
    return v;
}
#else
template <int CODE>
__device__ __forceinline__ int ck_idx(int v, int) { return v; }
#endif

// With -DK2D_PHASE_CLOCKS the step kernel adds up, per phase of a step, the cycles that lane 0 of every scene group spends
// in it (clock64 at the phase boundaries, one atomic add per boundary): k2d_phase_cycles reads the sums.  The phases:
enum { PH_GEOMETRY, PH_ACTUATORS, PH_JOINT_PRESTEP, PH_BOX_TEST, PH_NARROWPHASE, PH_RECORDS, PH_LEVELS, PH_WARM_START, PH_ITERATIONS,
       PH_INTEGRATE_CORRECT, PH_EPILOGUE, PH_MEMORY_RECORD_SOLVE, PH_LOAD, PH_STORE, PH_COUNT };
#ifdef K2D_PHASE_CLOCKS
__device__ unsigned long long k2d_phase_sums[PH_COUNT];
#define K2D_PHASE_BEGIN() long long ph_t = clock64()
#define K2D_PHASE_RESTART() ph_t = clock64()
#define K2D_PHASE(i) do { const long long ph_n = clock64(); if (lane == 0) atomicAdd(&k2d_phase_sums[i], (unsigned long long)(ph_n - ph_t)); ph_t = ph_n; } while (0)
#else
#define K2D_PHASE_BEGIN() do { } while (0)
#define K2D_PHASE_RESTART() do { } while (0)
#define K2D_PHASE(i) do { } while (0)
#endif

// ---------------------------------------------------------------- exact helpers
__device__ __forceinline__ float fmin_cmp(float a, float b) { return a < b ? a : b; }
__device__ __forceinline__ float fmax_cmp(float a, float b) { return a > b ? a : b; }
__device__ __forceinline__ float dot2(float ax, float ay, float bx, float by) { return __fmaf_rn(ax, bx, ay * by); }
__device__ __forceinline__ float cross2(float ax, float ay, float bx, float by) { return __fmaf_rn(ax, by, -(ay * bx)); }
__device__ __forceinline__ void rot2(float c, float s, float vx, float vy, float &ox, float &oy) {
    ox = __fmaf_rn(c, vx, -(s * vy));
    oy = __fmaf_rn(s, vx, c * vy);
}
__device__ __forceinline__ float4 ld4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ void st4(float *p, float a, float b, float c) { *reinterpret_cast<float4 *>(p) = make_float4(a, b, c, 0.0f); }
__device__ __forceinline__ bool finite_bits(float v) { return (__float_as_uint(v) & 0x7f800000u) != 0x7f800000u; }

// Sine and cosine: reduction by multiples of pi/2 with a three-part constant and FMA, then the
// Taylor polynomials of degree 9 (sine) and 10 (cosine) on [-pi/4, pi/4].  |error| < 4e-7.
__device__ __forceinline__ void sincos_spec(float th, float &c, float &s) {
    if (!(fabsf(th) <= 1.0e6f)) { c = __int_as_float(0x7fc00000); s = c; return; }
    float k = rintf(th * 0x1.45f306p-1f);
    float r = __fmaf_rn(-k, 0x1.921fb6p+0f, th);
    r = __fmaf_rn(-k, -0x1.777a5cp-25f, r);
    r = __fmaf_rn(-k, -0x1.ee59dap-50f, r);
    int q = ((int)k) & 3;
    float r2 = r * r;
    float ps = __fmaf_rn(0x1.71de3ap-19f, r2, -0x1.a01a02p-13f);
    ps = __fmaf_rn(ps, r2, 0x1.111112p-7f);
    ps = __fmaf_rn(ps, r2, -0x1.555556p-3f);
    float sp = __fmaf_rn(ps * r2, r, r);
    float pc = __fmaf_rn(-0x1.27e4fcp-22f, r2, 0x1.a01a02p-16f);
    pc = __fmaf_rn(pc, r2, -0x1.6c16c2p-10f);
    pc = __fmaf_rn(pc, r2, 0x1.555556p-5f);
    pc = __fmaf_rn(pc, r2, -0.5f);
    float cp = __fmaf_rn(pc, r2, 1.0f);
    float cc = (q & 1) ? sp : cp;      // |cos| source
    float ss = (q & 1) ? cp : sp;      // |sin| source
    c = (q == 1 || q == 2) ? -cc : cc;
    s = (q >= 2) ? -ss : ss;
}

// tanh(x) = sign(x) (1 - t) / (1 + t), t = exp(-2 min(|x|, 10)); exp by reduction with ln 2 in
// two parts and the degree-7 Taylor polynomial.  |error| < 4e-7.
__device__ __forceinline__ float tanh_spec(float x) {
    if (x != x) return x;
    float ax = fmin_cmp(fabsf(x), 10.0f);
    float y = -2.0f * ax;
    float k = rintf(y * 0x1.715476p+0f);
    float r = __fmaf_rn(-k, 0x1.62e4p-1f, y);
    r = __fmaf_rn(-k, 0x1.7f7d1cp-20f, r);
    float p = __fmaf_rn(0x1.a01a02p-13f, r, 0x1.6c16c2p-10f);
    p = __fmaf_rn(p, r, 0x1.111112p-7f);
    p = __fmaf_rn(p, r, 0x1.555556p-5f);
    p = __fmaf_rn(p, r, 0x1.555556p-3f);
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    float scale = __int_as_float((((int)k) + 127) << 23);
    float t = p * scale;
    float v = (1.0f - t) / (1.0f + t);
    return x < 0.0f ? -v : v;
}

// splitmix64 finaliser: level choice on auto-reset
__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL;
    z ^= z >> 27; z *= 0x94D049BB133111EBULL;
    z ^= z >> 31;
    return z;
}

// ---------------------------------------------------------------- group of G lanes
template <int G>
struct Group {
    unsigned mask;
    int lane, shift;
    __device__ __forceinline__ Group() {
        int wl = threadIdx.x & 31;
        shift = wl / G * G;
        lane = wl - shift;
        mask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << shift);
    }
    __device__ __forceinline__ void sync() const { __syncwarp(mask); }
    __device__ __forceinline__ unsigned ballot(bool p) const {
        unsigned b = __ballot_sync(mask, p) >> shift;
        return (G == 32) ? b : (b & ((1u << G) - 1u));
    }
    __device__ __forceinline__ int shfl(int v, int src) const { return __shfl_sync(mask, v, src, G); }
    __device__ __forceinline__ unsigned shflu(unsigned v, int src) const { return __shfl_sync(mask, v, src, G); }
    __device__ __forceinline__ float shflf(float v, int src) const { return __shfl_sync(mask, v, src, G); }
    __device__ __forceinline__ int max_int(int v) const { return __reduce_max_sync(mask, v); }
    __device__ __forceinline__ int sum_int(int v) const { return (int)__reduce_add_sync(mask, (unsigned)v); }
    __device__ __forceinline__ bool any(bool p) const { return __ballot_sync(mask, p) != 0; }
    __device__ __forceinline__ unsigned lanes_below() const { return (1u << lane) - 1u; }
};

// one manifold as the narrowphase leaves it
struct Manifold { float px, py, nx, ny, pen; };

// What the lane that owns a contact pair record keeps in registers for the whole step: the pair
// (packed word), the shared normal, the friction coefficient, the inverse masses and inertias of
// the two bodies, and the first manifold's lever-arm cross products, effective masses, target
// normal velocity and accumulated impulses.  The second manifold (polygon-polygon pairs only) is
// in the lane's shared-memory fields.
struct Rec {
    uint32_t ab;
    float nx, ny, mu, ma, mb, ia, ib;
    float rna, rnb, rta, rtb, massn, masst, target, accn, acct;
};
// memory form (overflow path)
struct RecM {
    uint32_t ab;
    float nx, ny, mu;
    float rna[2], rnb[2], rta[2], rtb[2], massn[2], masst[2], target[2], corr[2], accn[2], acct[2];
};

struct ContactConsts { float slop, rest_thr, alpha, beta; };

// ---- contact pre-step for one manifold of pair (a, b) with normal (nx, ny)
template <class SC>
__device__ __forceinline__ void prestep_manifold(int a, int b, float nx, float ny, float ma, float mb, float ia, float ib,
                                                 float px, float py, float pen, float er, const float *sm, const ContactConsts &cc,
                                                 float &rna, float &rnb, float &rta, float &rtb, float &massn, float &masst,
                                                 float &target, float &corr) {
    const float4 pa4 = ld4(sm + SC::BPOS + 4 * a), pb4 = ld4(sm + SC::BPOS + 4 * b);
    const float4 va4 = ld4(sm + SC::BVEL + 4 * a), vb4 = ld4(sm + SC::BVEL + 4 * b);
    const float rax = px - pa4.x, ray = py - pa4.y;
    const float rbx = px - pb4.x, rby = py - pb4.y;
    const float tx = -ny, ty = nx;
    rna = cross2(rax, ray, nx, ny); rnb = cross2(rbx, rby, nx, ny);
    rta = cross2(rax, ray, tx, ty); rtb = cross2(rbx, rby, tx, ty);
    float kn = ma + mb; kn = __fmaf_rn(ia * rna, rna, kn); kn = __fmaf_rn(ib * rnb, rnb, kn);
    float kt = ma + mb; kt = __fmaf_rn(ia * rta, rta, kt); kt = __fmaf_rn(ib * rtb, rtb, kt);
    // normal approach speed before warm starting
    float vn0 = dot2(nx, ny, vb4.x - va4.x, vb4.y - va4.y);
    vn0 = __fmaf_rn(vb4.z, rnb, vn0);
    vn0 = __fmaf_rn(-va4.z, rna, vn0);
    const float depth = fmax_cmp(pen - cc.slop, 0.0f);
    const float bounce = (vn0 < -cc.rest_thr) ? (-er * vn0) : 0.0f;
    massn = 1.0f / kn; masst = 1.0f / kt;
    target = bounce + cc.alpha * depth;
    corr = (cc.beta * depth) / (ma + mb);
}

// ---- one manifold's normal row then friction row on the velocities of its two bodies.
// MODE 0: apply the accumulated impulses (warm start); MODE 1: one solver iteration.
template <int MODE>
__device__ __forceinline__ void manifold_rows(float nx, float ny, float mu, float ma, float mb, float ia, float ib,
                                              float rna, float rnb, float rta, float rtb, float massn, float masst, float target,
                                              float &accn, float &acct,
                                              float &vax, float &vay, float &wa, float &vbx, float &vby, float &wb) {
    const float tx = -ny, ty = nx;
    const float wna = ia * rna, wnb = ib * rnb, wta = ia * rta, wtb = ib * rtb;
    float dn, dt_;
    if (MODE == 0) { dn = accn; }
    else {
        float vn = dot2(nx, ny, vbx - vax, vby - vay);
        vn = __fmaf_rn(wb, rnb, vn);
        vn = __fmaf_rn(-wa, rna, vn);
        const float lam = (target - vn) * massn;
        const float nw = fmax_cmp(accn + lam, 0.0f);
        dn = nw - accn; accn = nw;
    }
    {
        const float px = dn * nx, py = dn * ny;
        vax = __fmaf_rn(-ma, px, vax); vay = __fmaf_rn(-ma, py, vay); wa = __fmaf_rn(-wna, dn, wa);
        vbx = __fmaf_rn(mb, px, vbx); vby = __fmaf_rn(mb, py, vby); wb = __fmaf_rn(wnb, dn, wb);
    }
    if (MODE == 0) { dt_ = acct; }
    else {
        float vt = dot2(tx, ty, vbx - vax, vby - vay);
        vt = __fmaf_rn(wb, rtb, vt);
        vt = __fmaf_rn(-wa, rta, vt);
        const float lam = (-vt) * masst;
        const float lim = mu * accn;
        const float nw = fmax_cmp(fmin_cmp(acct + lam, lim), -lim);
        dt_ = nw - acct; acct = nw;
    }
    {
        const float px = dt_ * tx, py = dt_ * ty;
        vax = __fmaf_rn(-ma, px, vax); vay = __fmaf_rn(-ma, py, vay); wa = __fmaf_rn(-wta, dt_, wa);
        vbx = __fmaf_rn(mb, px, vbx); vby = __fmaf_rn(mb, py, vby); wb = __fmaf_rn(wtb, dt_, wb);
    }
}

// positional correction of one pair: each active manifold moves the two bodies apart along the normal
__device__ __forceinline__ void correct_pair(float *pos, int a, int b, unsigned amask, bool dyn_a, bool dyn_b,
                                             float nx, float ny, float ma, float mb, float corr0, float corr1) {
    float xa = pos[4 * a], ya = pos[4 * a + 1], xb = pos[4 * b], yb = pos[4 * b + 1];
    if (amask & 1u) {
        const float ca = ma * corr0, cb = mb * corr0;
        xa = __fmaf_rn(-ca, nx, xa); ya = __fmaf_rn(-ca, ny, ya);
        xb = __fmaf_rn(cb, nx, xb); yb = __fmaf_rn(cb, ny, yb);
    }
    if (amask & 2u) {
        const float ca = ma * corr1, cb = mb * corr1;
        xa = __fmaf_rn(-ca, nx, xa); ya = __fmaf_rn(-ca, ny, ya);
        xb = __fmaf_rn(cb, nx, xb); yb = __fmaf_rn(cb, ny, yb);
    }
    if (dyn_a) { pos[4 * a] = xa; pos[4 * a + 1] = ya; }
    if (dyn_b) { pos[4 * b] = xb; pos[4 * b + 1] = yb; }
}

// ---- angular row of a fixed joint or of a revolute joint beyond one of its limits (paper, "Fixed Joints",
// "Joint Limits"): j_r = (w_a - w_b + correction) / (1/I_a + 1/I_b), a loses j_r / I_a, b gains j_r / I_b.  A fixed
// joint's impulse is accumulated and warm-started; a limit only ever pushes back, applies no correction while the
// joint is already returning, and is not accumulated.  Returns the two angular velocities.  Out of line: most
// joints are plain revolute joints.
template <int MODE>
__device__ __noinline__ float2 angular_row(float *jr, float ia, float ib, float wa, float wb) {
    const float4 ang4 = ld4(jr + JR_ANG);      // kind this step, inverse angular mass, correction, accumulated impulse
    const int ang = __float_as_int(ang4.x);
    if (ang == 0) return make_float2(wa, wb);
    float lr;
    if (MODE == 0) {
        if (ang != 1) return make_float2(wa, wb);
        lr = ang4.w;
    } else {
        const float wrel = wa - wb;
        float v;
        if (ang == 1) v = wrel + ang4.z;
        else if (ang == 2) { v = (wrel < 0.0f) ? wrel : wrel + ang4.z; v = fmax_cmp(v, 0.0f); }
        else { v = (wrel > 0.0f) ? wrel : wrel + ang4.z; v = fmin_cmp(v, 0.0f); }
        lr = v * ang4.y;
        if (ang == 1) jr[JR_ACCR] = ang4.w + lr;
    }
    return make_float2(__fmaf_rn(-lr, ia, wa), __fmaf_rn(lr, ib, wb));
}

// ---- joints; the row of joint j is in shared memory.  MODE 0: warm start, 1: solver iteration,
// 2: positional correction, 3: motor
template <class SC, int MODE>
__device__ __forceinline__ void visit_joint(float *sm, uint32_t jab, int j, float motor_rho, int discrete = 0) {
    const int a = ck_idx<CK_BODY>(jab & 255, SC::N), b = ck_idx<CK_BODY>((jab >> 8) & 255, SC::N);
    const bool dyn_a = (jab >> 29) & 1u, dyn_b = (jab >> 30) & 1u;
    float *jr = sm + SC::JROW + kJointWords * j;
    if (MODE == 3) {
        const float av = sm[SC::ACT + ck_idx<CK_COUNT>((jab >> 16) & 255, kMaxActions)];
        // paper, "Action Space": continuous in [-1, 1], or multi-discrete codes 0 off, 1 forwards, 2 backwards at full power
        const float A = discrete ? (__float_as_int(av) == 1 ? 1.0f : (__float_as_int(av) == 2 ? -1.0f : 0.0f))
                                 : fmax_cmp(fmin_cmp(av, 1.0f), -1.0f);
        const float *jl = sm + SC::LVC + (SC::LV_JOINT - SC::LV_ELEN) + kJointLevelWords * j;
        const float speed = jl[5], power = jl[6];
        const float wa = sm[SC::BVEL + 4 * a + 2], wb = sm[SC::BVEL + 4 * b + 2];
        const float arg = __fmaf_rn(-speed, A, wa - wb) * motor_rho;
        const float jr_ = power * tanh_spec(arg);
        if (dyn_a) sm[SC::BVEL + 4 * a + 2] = __fmaf_rn(-jr_, sm[SC::BII + a], wa);
        if (dyn_b) sm[SC::BVEL + 4 * b + 2] = __fmaf_rn(jr_, sm[SC::BII + b], wb);
        return;
    }
    const float4 mi4 = ld4(jr + JR_MA);       // inverse masses and inertias of the two bodies
    const float ma = mi4.x, mb = mi4.y, ia = mi4.z, ib = mi4.w;
    if (MODE == 2) {
        const float cx = jr[JR_CX], cy = jr[JR_CY];
        if (dyn_a) { sm[SC::BPOS + 4 * a] = __fmaf_rn(ma, cx, sm[SC::BPOS + 4 * a]); sm[SC::BPOS + 4 * a + 1] = __fmaf_rn(ma, cy, sm[SC::BPOS + 4 * a + 1]); }
        if (dyn_b) { sm[SC::BPOS + 4 * b] = __fmaf_rn(-mb, cx, sm[SC::BPOS + 4 * b]); sm[SC::BPOS + 4 * b + 1] = __fmaf_rn(-mb, cy, sm[SC::BPOS + 4 * b + 1]); }
        return;
    }
    const float4 r4 = ld4(jr + JR_RAX);
    const float rax = r4.x, ray = r4.y, rbx = r4.z, rby = r4.w;
    const float4 va4 = ld4(sm + SC::BVEL + 4 * a), vb4 = ld4(sm + SC::BVEL + 4 * b);
    float vax = va4.x, vay = va4.y, wa = va4.z, vbx = vb4.x, vby = vb4.y, wb = vb4.z;
    float lx, ly;
    if (MODE == 0) { lx = jr[JR_ACCX]; ly = jr[JR_ACCY]; }
    else {
        const float4 k4 = ld4(jr + JR_I11), b4 = ld4(jr + JR_BX);
        const float2 acc = *reinterpret_cast<const float2 *>(jr + JR_ACCX);
        const float cx = __fmaf_rn(-wb, rby, vbx) - __fmaf_rn(-wa, ray, vax);
        const float cy = __fmaf_rn(wb, rbx, vby) - __fmaf_rn(wa, rax, vay);
        const float rx = -(cx + b4.x), ry = -(cy + b4.y);
        const float i11 = k4.x, i12 = k4.y, i22 = k4.z;
        lx = __fmaf_rn(i11, rx, i12 * ry);
        ly = __fmaf_rn(i12, rx, i22 * ry);
        *reinterpret_cast<float2 *>(jr + JR_ACCX) = make_float2(acc.x + lx, acc.y + ly);
    }
    wa = __fmaf_rn(-ia, cross2(rax, ray, lx, ly), wa);
    wb = __fmaf_rn(ib, cross2(rbx, rby, lx, ly), wb);
    if (jab >> 31) {      // fixed or limited joint: its angular row follows the point row
        const float2 w2 = angular_row<MODE>(jr, ia, ib, wa, wb);
        wa = w2.x; wb = w2.y;
    }
    if (dyn_a) st4(sm + SC::BVEL + 4 * a, __fmaf_rn(-ma, lx, vax), __fmaf_rn(-ma, ly, vay), wa);
    if (dyn_b) st4(sm + SC::BVEL + 4 * b, __fmaf_rn(mb, lx, vbx), __fmaf_rn(mb, ly, vby), wb);
}
// joints of one level touch disjoint movable bodies; levels in order keep the joint order
template <class SC, int G, int MODE>
__device__ __forceinline__ void sweep_joints(float *sm, uint32_t jab, int lane, int jlevel, int jmax, float motor_rho,
                                             int discrete = 0) {
    const unsigned mask = Group<G>().mask;
    if (SC::J == 0) return;
#pragma unroll 1
    for (int lvl = 1; lvl <= jmax; ++lvl) {
        if (jlevel == lvl) visit_joint<SC, MODE>(sm, jab, lane, motor_rho, discrete);
        __syncwarp(mask);
    }
}

// Accumulated impulses that pair record `wi` of the previous step left behind (255: the pair was not
// touching).  Records 0..G-1 live with lane wi (first manifold in its registers: old_n / old_t are the
// calling lane's own, fetched across lanes here, so every lane of the group must call; second manifold
// in its shared-memory fields), the next G / 2 records in the second-record fields of lane wi - G, later ones
// in the warm entries of the global scratch.
template <class SC, int G>
__device__ __forceinline__ void warm_lookup(const Group<G> &g, const float *sm, const uint32_t *ovf, int wi, float old_n, float old_t,
                                            int warm_start, float (&w)[4]) {
    wi = (wi == 255) ? 255 : ck_idx<CK_WARM>(wi, SC::NPAIRS);
    const int src = (wi < G) ? wi : 0;
    const float *lf = sm + SC::STG;
    w[0] = g.shflf(old_n, src); w[1] = g.shflf(old_t, src);
    w[2] = lf[LF_ACC2N * G + src]; w[3] = lf[LF_ACC2T * G + src];
    if (wi >= G && wi != 255) {
        if (wi < G + G / 2) {
            const float *o = lf + LF_COUNT * G + (wi - G);
            w[0] = o[OV_ACC0N * (G / 2)]; w[1] = o[OV_ACC0T * (G / 2)]; w[2] = o[OV_ACC1N * (G / 2)]; w[3] = o[OV_ACC1T * (G / 2)];
        } else {
            const uint32_t *wr = ovf + SC::SCRATCH_WARM + (size_t)wi * kWarmWords;
#pragma unroll
            for (int q = 0; q < 4; ++q) w[q] = __uint_as_float(wr[1 + q]);
        }
    }
    if (wi == 255 || !warm_start) { w[0] = 0.0f; w[1] = 0.0f; w[2] = 0.0f; w[3] = 0.0f; }
}

// Levels of nrec staged pairs by one lane with a per-body table (used when there are more pairs than
// lanes): a pair's level is one more than the highest level of an earlier pair sharing a movable body.
// The packed pair words of pairs 0..G-1 are in the stage fields, of the next G / 2 in the second-record
// fields, of later ones in global scratch; the level goes into bits 19.. of each word.
template <class SC, int G>
__device__ __noinline__ int levels_by_one_lane(uint32_t *smu, uint32_t *ovf, int nrec) {
    uint8_t *bl = reinterpret_cast<uint8_t *>(smu + SC::SURV);   // the survivor list is no longer needed
    int cmax = 0;
    for (int i = 0; i < SC::N; ++i) bl[i] = 0;
    for (int k = 0; k < nrec; ++k) {
        uint32_t *w = (k < G) ? (smu + SC::STG + S_AB * G + k)
                    : (k < G + G / 2) ? (smu + SC::STG + LF_COUNT * G + ovs(S_AB) * (G / 2) + (k - G)) : (ovf + (size_t)ck_idx<CK_RECORD>(k, SC::NPAIRS) * kRecWords + S_AB);
        const uint32_t ab = *w;
        const int a = ck_idx<CK_BODY>(ab & 31, SC::N), b = ck_idx<CK_BODY>((ab >> 5) & 31, SC::N);
        int lvl = 1;
        if ((ab >> 26) & 1u) lvl = max(lvl, bl[a] + 1);
        if ((ab >> 27) & 1u) lvl = max(lvl, bl[b] + 1);
        if ((ab >> 26) & 1u) bl[a] = (uint8_t)lvl;
        if ((ab >> 27) & 1u) bl[b] = (uint8_t)lvl;
        *w = ab | ((uint32_t)ck_idx<CK_SOLVER_LEVEL>(lvl, 128) << 19);
        cmax = max(cmax, lvl);
    }
    return cmax;
}

// ================================================================ overflow path (cold code)
// A scene with more touching pairs than lanes (nrec > G) solves this step's contacts from memory
// records in global scratch, one loop over records per level, with the same row arithmetic.
__device__ __forceinline__ void recm_load(const uint32_t *r, RecM &c) {
    c.ab = r[R_AB]; c.nx = __uint_as_float(r[R_NX]); c.ny = __uint_as_float(r[R_NY]); c.mu = __uint_as_float(r[R_MU]);
#pragma unroll
    for (int mi = 0; mi < 2; ++mi) {
        const uint32_t *m = r + R_M0 + mi * M_WORDS;
        c.rna[mi] = __uint_as_float(m[M_RNA]); c.rnb[mi] = __uint_as_float(m[M_RNB]);
        c.rta[mi] = __uint_as_float(m[M_RTA]); c.rtb[mi] = __uint_as_float(m[M_RTB]);
        c.massn[mi] = __uint_as_float(m[M_MASSN]); c.masst[mi] = __uint_as_float(m[M_MASST]);
        c.target[mi] = __uint_as_float(m[M_TARGET]); c.corr[mi] = __uint_as_float(m[M_CORR]);
        c.accn[mi] = __uint_as_float(m[M_ACCN]); c.acct[mi] = __uint_as_float(m[M_ACCT]);
    }
}
__device__ __forceinline__ void recm_store(uint32_t *r, const RecM &c) {
    r[R_AB] = c.ab; r[R_NX] = __float_as_uint(c.nx); r[R_NY] = __float_as_uint(c.ny); r[R_MU] = __float_as_uint(c.mu);
#pragma unroll
    for (int mi = 0; mi < 2; ++mi) {
        uint32_t *m = r + R_M0 + mi * M_WORDS;
        m[M_RNA] = __float_as_uint(c.rna[mi]); m[M_RNB] = __float_as_uint(c.rnb[mi]);
        m[M_RTA] = __float_as_uint(c.rta[mi]); m[M_RTB] = __float_as_uint(c.rtb[mi]);
        m[M_MASSN] = __float_as_uint(c.massn[mi]); m[M_MASST] = __float_as_uint(c.masst[mi]);
        m[M_TARGET] = __float_as_uint(c.target[mi]); m[M_CORR] = __float_as_uint(c.corr[mi]);
        m[M_ACCN] = __float_as_uint(c.accn[mi]); m[M_ACCT] = __float_as_uint(c.acct[mi]);
    }
}

template <class SC, int G, int MODE>
__device__ __forceinline__ void slow_sweep_pairs(float *sm, uint32_t *ovf, int nrec, int cmax) {
    Group<G> g;
    for (int lvl = 1; lvl <= cmax; ++lvl) {
        for (int k = g.lane; k < nrec; k += G) {
            uint32_t *r = ovf + (size_t)ck_idx<CK_RECORD>(k, SC::NPAIRS) * kRecWords;
            if (((r[R_AB] >> 19) & 127u) != (unsigned)lvl) continue;
            RecM c;
            recm_load(r, c);
            const int a = ck_idx<CK_BODY>(c.ab & 31, SC::N), b = ck_idx<CK_BODY>((c.ab >> 5) & 31, SC::N);
            const unsigned amask = (c.ab >> 10) & 3u;
            const bool dyn_a = (c.ab >> 26) & 1u, dyn_b = (c.ab >> 27) & 1u;
            const float ma = sm[SC::BIM + a], mb = sm[SC::BIM + b];
            if (MODE == 2) { correct_pair(sm + SC::BPOS, a, b, amask, dyn_a, dyn_b, c.nx, c.ny, ma, mb, c.corr[0], c.corr[1]); continue; }
            const float ia = sm[SC::BII + a], ib = sm[SC::BII + b];
            const float4 va4 = ld4(sm + SC::BVEL + 4 * a), vb4 = ld4(sm + SC::BVEL + 4 * b);
            float vax = va4.x, vay = va4.y, wa = va4.z, vbx = vb4.x, vby = vb4.y, wb = vb4.z;
#pragma unroll
            for (int mi = 0; mi < 2; ++mi) {
                if (amask & (1u << mi)) {
                    manifold_rows<MODE>(c.nx, c.ny, c.mu, ma, mb, ia, ib, c.rna[mi], c.rnb[mi], c.rta[mi], c.rtb[mi], c.massn[mi], c.masst[mi],
                                        c.target[mi], c.accn[mi], c.acct[mi], vax, vay, wa, vbx, vby, wb);
                    if (MODE == 1) {
                        r[R_M0 + mi * M_WORDS + M_ACCN] = __float_as_uint(c.accn[mi]);
                        r[R_M0 + mi * M_WORDS + M_ACCT] = __float_as_uint(c.acct[mi]);
                    }
                }
            }
            if (dyn_a) st4(sm + SC::BVEL + 4 * a, vax, vay, wa);
            if (dyn_b) st4(sm + SC::BVEL + 4 * b, vbx, vby, wb);
        }
        g.sync();
    }
}

// ---- batched contact solve (paper, "Parallelised Computation and Batched Impulse Resolution"): the i-th active manifold
// (canonical order) belongs to batch i mod n_batches; the rows of a batch are all solved against the velocities the batch
// starts with, then applied; batches follow one another.  One iteration over the memory records in scratch; the warm
// entries of the scratch, free between the pre-step and the end of the step, hold per record the rank of its first
// manifold and the impulses to apply.
__device__ __forceinline__ void apply_impulse(float d, float dx, float dy, float ma, float mb, float lev_a, float lev_b,
                                              float &vax, float &vay, float &wa, float &vbx, float &vby, float &wb) {
    const float px = d * dx, py = d * dy;
    vax = __fmaf_rn(-ma, px, vax); vay = __fmaf_rn(-ma, py, vay); wa = __fmaf_rn(-lev_a, d, wa);
    vbx = __fmaf_rn(mb, px, vbx); vby = __fmaf_rn(mb, py, vby); wb = __fmaf_rn(lev_b, d, wb);
}
template <class SC, int G>
__device__ __noinline__ void slow_batched_iteration(float *sm, uint32_t *ovf, int nrec, int cmax, int nman, int n_batches) {
    Group<G> g;
    uint32_t *aux = ovf + SC::SCRATCH_WARM;
    const int nb_used = nman < n_batches ? nman : n_batches;
    for (int bt = 0; bt < nb_used; ++bt) {
        // every row of the batch against the velocities as they stand: impulses and accumulated impulses, no velocity is written
        for (int k = g.lane; k < nrec; k += G) {
            uint32_t *r = ovf + (size_t)ck_idx<CK_RECORD>(k, SC::NPAIRS) * kRecWords;
            RecM c;
            recm_load(r, c);
            const int a = ck_idx<CK_BODY>(c.ab & 31, SC::N), b = ck_idx<CK_BODY>((c.ab >> 5) & 31, SC::N);
            const unsigned amask = (c.ab >> 10) & 3u;
            const int rank0 = (int)aux[kWarmWords * k];
            const float ma = sm[SC::BIM + a], mb = sm[SC::BIM + b], ia = sm[SC::BII + a], ib = sm[SC::BII + b];
            const float4 va4 = ld4(sm + SC::BVEL + 4 * a), vb4 = ld4(sm + SC::BVEL + 4 * b);
#pragma unroll 1
            for (int mi = 0; mi < 2; ++mi) {
                if (!(amask & (1u << mi))) continue;
                const int rank = rank0 + ((mi == 1 && (amask & 1u)) ? 1 : 0);
                if (rank % n_batches != bt) continue;
                float vax = va4.x, vay = va4.y, wa = va4.z, vbx = vb4.x, vby = vb4.y, wb = vb4.z;
                const float old_n = c.accn[mi], old_t = c.acct[mi];
                manifold_rows<1>(c.nx, c.ny, c.mu, ma, mb, ia, ib, c.rna[mi], c.rnb[mi], c.rta[mi], c.rtb[mi], c.massn[mi], c.masst[mi],
                                 c.target[mi], c.accn[mi], c.acct[mi], vax, vay, wa, vbx, vby, wb);
                r[R_M0 + mi * M_WORDS + M_ACCN] = __float_as_uint(c.accn[mi]);
                r[R_M0 + mi * M_WORDS + M_ACCT] = __float_as_uint(c.acct[mi]);
                aux[kWarmWords * k + 1 + 2 * mi] = __float_as_uint(c.accn[mi] - old_n);
                aux[kWarmWords * k + 2 + 2 * mi] = __float_as_uint(c.acct[mi] - old_t);
            }
        }
        g.sync();
        // the batch's impulses, applied in canonical order per body: level by level
        for (int lvl = 1; lvl <= cmax; ++lvl) {
            for (int k = g.lane; k < nrec; k += G) {
                const uint32_t *r = ovf + (size_t)ck_idx<CK_RECORD>(k, SC::NPAIRS) * kRecWords;
                const uint32_t ab = r[R_AB];
                if (((ab >> 19) & 127u) != (unsigned)lvl) continue;
                const unsigned amask = (ab >> 10) & 3u;
                const int rank0 = (int)aux[kWarmWords * k];
                const bool in0 = (amask & 1u) && rank0 % n_batches == bt;
                const bool in1 = (amask & 2u) && (rank0 + ((amask & 1u) ? 1 : 0)) % n_batches == bt;
                if (!in0 && !in1) continue;
                const int a = ck_idx<CK_BODY>(ab & 31, SC::N), b = ck_idx<CK_BODY>((ab >> 5) & 31, SC::N);
                const float nx = __uint_as_float(r[R_NX]), ny = __uint_as_float(r[R_NY]);
                const float ma = sm[SC::BIM + a], mb = sm[SC::BIM + b], ia = sm[SC::BII + a], ib = sm[SC::BII + b];
                const float4 va4 = ld4(sm + SC::BVEL + 4 * a), vb4 = ld4(sm + SC::BVEL + 4 * b);
                float vax = va4.x, vay = va4.y, wa = va4.z, vbx = vb4.x, vby = vb4.y, wb = vb4.z;
#pragma unroll 1
                for (int mi = 0; mi < 2; ++mi) {
                    if (!(mi ? in1 : in0)) continue;
                    const uint32_t *m = r + R_M0 + mi * M_WORDS;
                    const float rna = __uint_as_float(m[M_RNA]), rnb = __uint_as_float(m[M_RNB]), rta = __uint_as_float(m[M_RTA]), rtb = __uint_as_float(m[M_RTB]);
                    const float dn = __uint_as_float(aux[kWarmWords * k + 1 + 2 * mi]), dt_ = __uint_as_float(aux[kWarmWords * k + 2 + 2 * mi]);
                    apply_impulse(dn, nx, ny, ma, mb, ia * rna, ib * rnb, vax, vay, wa, vbx, vby, wb);
                    apply_impulse(dt_, -ny, nx, ma, mb, ia * rta, ib * rtb, vax, vay, wa, vbx, vby, wb);
                }
                if ((ab >> 26) & 1u) st4(sm + SC::BVEL + 4 * a, vax, vay, wa);
                if ((ab >> 27) & 1u) st4(sm + SC::BVEL + 4 * b, vbx, vby, wb);
            }
            g.sync();
        }
    }
}

// ---- all solver iterations of a scene in the batched order (paper, "Parallelised Computation and Batched Impulse Resolution"),
// from the lanes' own records: the rank of a manifold among the scene's active manifolds (pair order, slot 0 then 1) gives
// its batch, rank mod n_batches; per batch every row is solved against the velocities as they stand (its lane's private
// copy), then the batch's impulses are applied level by level, which is the canonical order on every body.  For scenes
// without second records.  Returns the accumulated impulses of the lane's first manifold.  Out of line: the default order
// is the sequential one.
template <class SC, int G>
__device__ __noinline__ float2 batched_iterations(float *sm, Rec rec, uint32_t jab, int jlevel, int jmax, int cmax, int clevel,
                                                  int solver_iters, float motor_rho, int n_batches) {
    Group<G> g;
    const int lane = g.lane;
    const uint32_t ab = rec.ab;
    const int a = ck_idx<CK_BODY>(ab & 31, SC::N), b = ck_idx<CK_BODY>((ab >> 5) & 31, SC::N);
    const unsigned amask = (ab >> 10) & 3u;
    float *lf = sm + SC::STG + lane;                 // this lane's fields: field f at lf[f * G]
    const unsigned has0 = g.ballot(amask & 1u), has1 = g.ballot(amask & 2u);
    const int rank0 = __popc(has0 & g.lanes_below()) + __popc(has1 & g.lanes_below());
    const int b0 = (amask & 1u) ? rank0 % n_batches : -1;
    const int b1 = (amask & 2u) ? (rank0 + (int)(amask & 1u)) % n_batches : -1;
#pragma unroll 1
    for (int it = 0; it < solver_iters; ++it) {
        sweep_joints<SC, G, 1>(sm, jab, lane, jlevel, jmax, motor_rho);
#pragma unroll 1
        for (int bt = 0; bt < n_batches; ++bt) {
            const bool in0 = b0 == bt, in1 = b1 == bt;
            if (!g.any(in0 || in1)) break;      // batches are filled in order: the first empty one ends the sweep
            float d0n = 0.0f, d0t = 0.0f, d1n = 0.0f, d1t = 0.0f;
            if (in0 || in1) {
                const float4 va4 = ld4(sm + SC::BVEL + 4 * a), vb4 = ld4(sm + SC::BVEL + 4 * b);
                if (in0) {
                    float vax = va4.x, vay = va4.y, wa = va4.z, vbx = vb4.x, vby = vb4.y, wb = vb4.z;
                    const float old_n = rec.accn, old_t = rec.acct;
                    manifold_rows<1>(rec.nx, rec.ny, rec.mu, rec.ma, rec.mb, rec.ia, rec.ib, rec.rna, rec.rnb, rec.rta, rec.rtb,
                                     rec.massn, rec.masst, rec.target, rec.accn, rec.acct, vax, vay, wa, vbx, vby, wb);
                    d0n = rec.accn - old_n; d0t = rec.acct - old_t;
                }
                if (in1) {
                    float vax = va4.x, vay = va4.y, wa = va4.z, vbx = vb4.x, vby = vb4.y, wb = vb4.z;
                    const float old_n = lf[LF_ACC2N * G], old_t = lf[LF_ACC2T * G];
                    float accn = old_n, acct = old_t;
                    manifold_rows<1>(rec.nx, rec.ny, rec.mu, rec.ma, rec.mb, rec.ia, rec.ib, lf[M2_RNA * G], lf[M2_RNB * G], lf[M2_RTA * G],
                                     lf[M2_RTB * G], lf[M2_MASSN * G], lf[M2_MASST * G], lf[M2_TARGET * G], accn, acct, vax, vay, wa, vbx, vby, wb);
                    lf[LF_ACC2N * G] = accn; lf[LF_ACC2T * G] = acct;
                    d1n = accn - old_n; d1t = acct - old_t;
                }
            }
            g.sync();
#pragma unroll 1
            for (int lvl = 1; lvl <= cmax; ++lvl) {
                if (clevel == lvl && (in0 || in1)) {
                    const float4 va4 = ld4(sm + SC::BVEL + 4 * a), vb4 = ld4(sm + SC::BVEL + 4 * b);
                    float vax = va4.x, vay = va4.y, wa = va4.z, vbx = vb4.x, vby = vb4.y, wb = vb4.z;
                    if (in0) {
                        apply_impulse(d0n, rec.nx, rec.ny, rec.ma, rec.mb, rec.ia * rec.rna, rec.ib * rec.rnb, vax, vay, wa, vbx, vby, wb);
                        apply_impulse(d0t, -rec.ny, rec.nx, rec.ma, rec.mb, rec.ia * rec.rta, rec.ib * rec.rtb, vax, vay, wa, vbx, vby, wb);
                    }
                    if (in1) {
                        apply_impulse(d1n, rec.nx, rec.ny, rec.ma, rec.mb, rec.ia * lf[M2_RNA * G], rec.ib * lf[M2_RNB * G], vax, vay, wa, vbx, vby, wb);
                        apply_impulse(d1t, -rec.ny, rec.nx, rec.ma, rec.mb, rec.ia * lf[M2_RTA * G], rec.ib * lf[M2_RTB * G], vax, vay, wa, vbx, vby, wb);
                    }
                    if ((ab >> 26) & 1u) st4(sm + SC::BVEL + 4 * a, vax, vay, wa);
                    if ((ab >> 27) & 1u) st4(sm + SC::BVEL + 4 * b, vbx, vby, wb);
                }
                g.sync();
            }
        }
    }
    return make_float2(rec.accn, rec.acct);
}

// Records from the staged manifolds (the first G in shared memory, the rest already in scratch),
// their levels, warm start and all solver iterations, joints included.  old_n / old_t: this lane's
// first-manifold accumulated impulses of the previous step.  Returns the highest contact level.
template <class SC, int G>
__device__ __noinline__ int slow_solve(float *sm, uint32_t *ovf, int nrec, uint32_t jab, int jlevel, int jmax,
                                       int solver_iters, int warm_start, float motor_rho, float old_n, float old_t, ContactConsts cc, int n_batches) {
    Group<G> g;
    const int lane = g.lane;
    uint32_t *smu = reinterpret_cast<uint32_t *>(sm);
    const uint8_t *widx = reinterpret_cast<const uint8_t *>(smu + SC::WIDX);
    int cmax = 0;
    if (lane == 0) cmax = levels_by_one_lane<SC, G>(smu, ovf, nrec);
    __threadfence_block();
    g.sync();
    cmax = g.shfl(cmax, 0);
    // the staged manifolds of the first G + G / 2 pairs join the others in scratch
    {
        uint32_t *r = ovf + (size_t)lane * kRecWords, *r2 = ovf + (size_t)(G + lane) * kRecWords;
#pragma unroll
        for (int f = 0; f < kStageWords; ++f) {
            if (lane < nrec) r[f] = smu[SC::STG + f * G + lane];
            if (lane < G / 2 && G + lane < nrec) r2[f] = smu[SC::STG + LF_COUNT * G + ovs(f) * (G / 2) + lane];
        }
    }
    g.sync();
    // pre-step of every pair; accumulated impulses of the previous step come from the lane that
    // owned the pair then (first manifold in its registers, second in its shared-memory fields)
    // or from the warm entries in scratch
    for (int base = 0; base < nrec; base += G) {
        const int k = base + lane;
        const bool valid = k < nrec;
        uint32_t *r = ovf + (size_t)(valid ? k : 0) * kRecWords;
        uint32_t ab = 0u;
        int wi = 255;
        if (valid) { ab = r[S_AB]; wi = widx[ck_idx<CK_PAIR>((ab >> 12) & 127, SC::NPAIRS)]; }
        float w[4];
        warm_lookup<SC, G>(g, sm, ovf, wi, old_n, old_t, warm_start, w);
        if (valid) {
            RecM c;
            c.ab = ab; c.nx = __uint_as_float(r[S_NX]); c.ny = __uint_as_float(r[S_NY]);
            const float pt[6] = { __uint_as_float(r[S_PX0]), __uint_as_float(r[S_PY0]), __uint_as_float(r[S_PEN0]),
                                  __uint_as_float(r[S_PX1]), __uint_as_float(r[S_PY1]), __uint_as_float(r[S_PEN1]) };
            const int a = ck_idx<CK_BODY>(ab & 31, SC::N), b = ck_idx<CK_BODY>((ab >> 5) & 31, SC::N);
            const float ma = sm[SC::BIM + a], mb = sm[SC::BIM + b], ia = sm[SC::BII + a], ib = sm[SC::BII + b];
            const float fra = sm[SC::BFR + a], frb = sm[SC::BFR + b];
            const float er = fmin_cmp(sm[SC::BRE + a], sm[SC::BRE + b]);
            c.mu = sqrtf(__fmaf_rn(fra, fra, frb * frb));
#pragma unroll
            for (int mi = 0; mi < 2; ++mi) {
                if ((ab >> 10) & (1u << mi)) {
                    prestep_manifold<SC>(a, b, c.nx, c.ny, ma, mb, ia, ib, pt[3 * mi], pt[3 * mi + 1], pt[3 * mi + 2], er, sm, cc,
                                         c.rna[mi], c.rnb[mi], c.rta[mi], c.rtb[mi], c.massn[mi], c.masst[mi], c.target[mi], c.corr[mi]);
                    c.accn[mi] = w[2 * mi]; c.acct[mi] = w[2 * mi + 1];
                } else {
                    c.rna[mi] = 0.0f; c.rnb[mi] = 0.0f; c.rta[mi] = 0.0f; c.rtb[mi] = 0.0f; c.massn[mi] = 0.0f; c.masst[mi] = 0.0f;
                    c.target[mi] = 0.0f; c.corr[mi] = 0.0f; c.accn[mi] = 0.0f; c.acct[mi] = 0.0f;
                }
            }
            recm_store(r, c);
        }
    }
    g.sync();
    int nman = 0;
    if (n_batches > 0) {
        // rank of every record's first manifold among the active manifolds, in canonical order
        if (lane == 0) {
            for (int k = 0; k < nrec; ++k) {
                ovf[SC::SCRATCH_WARM + kWarmWords * k] = (uint32_t)nman;
                nman += __popc((ovf[(size_t)k * kRecWords + R_AB] >> 10) & 3u);
            }
        }
        g.sync();
        nman = g.shfl(nman, 0);
    }
    slow_sweep_pairs<SC, G, 0>(sm, ovf, nrec, cmax);
    sweep_joints<SC, G, 0>(sm, jab, lane, jlevel, jmax, motor_rho);
    for (int it = 0; it < solver_iters; ++it) {
        sweep_joints<SC, G, 1>(sm, jab, lane, jlevel, jmax, motor_rho);
        if (nman > n_batches) slow_batched_iteration<SC, G>(sm, ovf, nrec, cmax, nman, n_batches);     // else one row per batch: the sequential sweep
        else slow_sweep_pairs<SC, G, 1>(sm, ovf, nrec, cmax);
    }
    return cmax;
}

template <class SC, int G>
__device__ __noinline__ void slow_correct(float *sm, uint32_t *ovf, int nrec, int cmax) {
    slow_sweep_pairs<SC, G, 2>(sm, ovf, nrec, cmax);
}

// End of an overflow step: every pair's accumulated impulses become warm entries in scratch and the
// pair index table learns where they are; returns the number of active manifolds.
template <class SC, int G>
__device__ __noinline__ int slow_finish(float *sm, uint32_t *ovf, int nrec) {
    Group<G> g;
    uint8_t *widx = reinterpret_cast<uint8_t *>(reinterpret_cast<uint32_t *>(sm) + SC::WIDX);
    int nman = 0;
    for (int k = g.lane; k < nrec; k += G) {
        const uint32_t *r = ovf + (size_t)ck_idx<CK_RECORD>(k, SC::NPAIRS) * kRecWords;
        uint32_t *wr = ovf + SC::SCRATCH_WARM + (size_t)k * kWarmWords;
        const uint32_t ab = r[R_AB];
        const int p = (ab >> 12) & 127;
        const unsigned am = (ab >> 10) & 3u;
        wr[0] = (uint32_t)p;
        wr[1] = (am & 1u) ? r[R_M0 + M_ACCN] : 0u;
        wr[2] = (am & 1u) ? r[R_M0 + M_ACCT] : 0u;
        wr[3] = (am & 2u) ? r[R_M0 + M_WORDS + M_ACCN] : 0u;
        wr[4] = (am & 2u) ? r[R_M0 + M_WORDS + M_ACCT] : 0u;
        widx[ck_idx<CK_PAIR>(p, SC::NPAIRS)] = (uint8_t)k;
        nman += __popc(am);
    }
    nman = g.sum_int(nman);
    g.sync();
    return nman;
}

// Launch boundaries: warm entries G + G / 2 .. between the state record and the scratch.
template <class SC, int G>
__device__ __noinline__ void warm_in(float *sm, uint32_t *ovf, const uint32_t *st_warm, int nwarm) {
    Group<G> g;
    uint8_t *widx = reinterpret_cast<uint8_t *>(reinterpret_cast<uint32_t *>(sm) + SC::WIDX);
    for (int k = G + G / 2 + g.lane; k < nwarm; k += G) {
        uint32_t *wr = ovf + SC::SCRATCH_WARM + (size_t)k * kWarmWords;
#pragma unroll
        for (int q = 0; q < kWarmWords; ++q) wr[q] = __ldcg(st_warm + kWarmWords * k + q);
        widx[ck_idx<CK_PAIR>((int)wr[0], SC::NPAIRS)] = (uint8_t)k;
    }
}
template <class SC, int G>
__device__ __noinline__ void warm_out(const uint32_t *ovf, uint32_t *st_warm, int nwarm) {
    Group<G> g;
    for (int k = G + G / 2 + g.lane; k < nwarm; k += G) {
        const uint32_t *wr = ovf + SC::SCRATCH_WARM + (size_t)k * kWarmWords;
#pragma unroll
        for (int q = 0; q < kWarmWords; ++q) st_warm[kWarmWords * k + q] = wr[q];
    }
}

// ---- one visit of the calling lane's second record (pair number G + lane of a scene with more than G
// touching pairs), which is in memory form in the lane's shared-memory fields.  MODE as for the first record.
template <class SC, int G, int MODE>
__device__ __noinline__ void visit_second(float *sm) {
    float *ov = sm + SC::STG + LF_COUNT * G + Group<G>().lane;
    constexpr int H = G / 2;
    const uint32_t ab = __float_as_uint(ov[R_AB * H]);
    const int a = ck_idx<CK_BODY>(ab & 31, SC::N), b = ck_idx<CK_BODY>((ab >> 5) & 31, SC::N);
    const unsigned amask = (ab >> 10) & 3u;
    const bool dyn_a = (ab >> 26) & 1u, dyn_b = (ab >> 27) & 1u;
    const float nx = ov[R_NX * H], ny = ov[R_NY * H];
    const float ma = sm[SC::BIM + a], mb = sm[SC::BIM + b];
    if (MODE == 2) {
        correct_pair(sm + SC::BPOS, a, b, amask, dyn_a, dyn_b, nx, ny, ma, mb, ov[(R_M0 + M_CORR) * H], ov[(R_M0 + M_WORDS + M_CORR) * H]);
        return;
    }
    const float ia = sm[SC::BII + a], ib = sm[SC::BII + b], mu = ov[R_MU * H];
    const float4 va4 = ld4(sm + SC::BVEL + 4 * a), vb4 = ld4(sm + SC::BVEL + 4 * b);
    float vax = va4.x, vay = va4.y, wa = va4.z, vbx = vb4.x, vby = vb4.y, wb = vb4.z;
#pragma unroll 1
    for (int mi = 0; mi < 2; ++mi) {
        if (amask & (1u << mi)) {
            float *m = ov + (R_M0 + mi * M_WORDS) * H;
            float accn = m[M_ACCN * H], acct = m[M_ACCT * H];
            manifold_rows<MODE>(nx, ny, mu, ma, mb, ia, ib, m[M_RNA * H], m[M_RNB * H], m[M_RTA * H], m[M_RTB * H],
                                m[M_MASSN * H], m[M_MASST * H], m[M_TARGET * H], accn, acct, vax, vay, wa, vbx, vby, wb);
            if (MODE == 1) { m[M_ACCN * H] = accn; m[M_ACCT * H] = acct; }
        }
    }
    if (dyn_a) st4(sm + SC::BVEL + 4 * a, vax, vay, wa);
    if (dyn_b) st4(sm + SC::BVEL + 4 * b, vbx, vby, wb);
}

// Second records, first half: the accumulated impulses the staged pair G + lane carried out of the
// previous step, parked in four of the lane's second-record fields that are free until the record is built.
template <class SC, int G>
__device__ __noinline__ void second_lookup(float *sm, const uint32_t *ovf, int nrec, float old_n, float old_t, int warm_start) {
    const Group<G> g;
    constexpr int H = G / 2;
    float *ov = sm + SC::STG + LF_COUNT * G + g.lane;
    const uint8_t *widx = reinterpret_cast<const uint8_t *>(reinterpret_cast<const uint32_t *>(sm) + SC::WIDX);
    const bool mine2 = g.lane < H && G + g.lane < nrec;
    int wi2 = 255;
    if (mine2) wi2 = widx[ck_idx<CK_PAIR>((__float_as_uint(ov[ovs(S_AB) * H]) >> 12) & 127, SC::NPAIRS)];
    float w2[4];
    warm_lookup<SC, G>(g, sm, ovf, wi2, old_n, old_t, warm_start, w2);
    if (mine2) {
#pragma unroll
        for (int q = 0; q < 4; ++q) ov[(R_M0 + M_WORDS + q) * H] = w2[q];
    }
}
// Second half, after every lane has read what it needs from other lanes: the record is built in place.
// Returns its level | its number of active manifolds << 8 (0 for a lane without a second record).
template <class SC, int G>
__device__ __noinline__ unsigned second_build(float *sm, int nrec, ContactConsts cc) {
    const int lane = Group<G>().lane;
    constexpr int H = G / 2;
    if (!(lane < H && G + lane < nrec)) return 0u;
    float *ov = sm + SC::STG + LF_COUNT * G + lane;
    const uint32_t ab2 = __float_as_uint(ov[ovs(S_AB) * H]);
    const int a2 = ck_idx<CK_BODY>(ab2 & 31, SC::N), b2 = ck_idx<CK_BODY>((ab2 >> 5) & 31, SC::N);
    const float nx2 = ov[ovs(S_NX) * H], ny2 = ov[ovs(S_NY) * H];
    const float pt2[6] = { ov[ovs(S_PX0) * H], ov[ovs(S_PY0) * H], ov[ovs(S_PEN0) * H], ov[ovs(S_PX1) * H], ov[ovs(S_PY1) * H], ov[ovs(S_PEN1) * H] };
    float w2[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) w2[q] = ov[(R_M0 + M_WORDS + q) * H];
    const float ma = sm[SC::BIM + a2], mb = sm[SC::BIM + b2], ia = sm[SC::BII + a2], ib = sm[SC::BII + b2];
    const float fra = sm[SC::BFR + a2], frb = sm[SC::BFR + b2];
    const float er2 = fmin_cmp(sm[SC::BRE + a2], sm[SC::BRE + b2]);
    ov[R_MU * H] = sqrtf(__fmaf_rn(fra, fra, frb * frb));
#pragma unroll 1
    for (int mi = 0; mi < 2; ++mi) {
        float rna = 0.0f, rnb = 0.0f, rta = 0.0f, rtb = 0.0f, massn = 0.0f, masst = 0.0f, target = 0.0f, corr = 0.0f, an = 0.0f, at = 0.0f;
        if ((ab2 >> 10) & (1u << mi)) {
            prestep_manifold<SC>(a2, b2, nx2, ny2, ma, mb, ia, ib, pt2[3 * mi], pt2[3 * mi + 1], pt2[3 * mi + 2], er2, sm, cc,
                                 rna, rnb, rta, rtb, massn, masst, target, corr);
            an = w2[2 * mi]; at = w2[2 * mi + 1];
        }
        float *m = ov + (R_M0 + mi * M_WORDS) * H;
        m[M_RNA * H] = rna; m[M_RNB * H] = rnb; m[M_RTA * H] = rta; m[M_RTB * H] = rtb;
        m[M_MASSN * H] = massn; m[M_MASST * H] = masst; m[M_TARGET * H] = target; m[M_CORR * H] = corr;
        m[M_ACCN * H] = an; m[M_ACCT * H] = at;
    }
    return ((ab2 >> 19) & 127u) | ((unsigned)__popc((ab2 >> 10) & 3u) << 8);
}

// ================================================================ rarely run code, kept out of line
// so that the code a step normally runs stays small
// level constants into shared memory; returns the packed word of joint number `lane` (0 beyond the last joint)
template <class SC, int G>
__device__ __noinline__ uint32_t load_level_consts(uint32_t *smu, const uint32_t *lv) {
    const int lane = Group<G>().lane;
    // all loads are asked for before the first of them is stored, so that the group waits for memory once
    constexpr int KN = (SC::N + G - 1) / G, KL = (SC::LVC_WORDS + G - 1) / G, KC = (SC::C + G - 1) / G, KM = (SC::MASKW + G - 1) / G;
    uint32_t cim[KN], cii[KN], cfr[KN], cre[KN], cfl[KN], lvc[KL], rad[KC], msk[KM];
#pragma unroll
    for (int k = 0; k < KN; ++k) {
        const int i = lane + k * G; const bool in = i < SC::N;
        cim[k] = in ? __ldg(lv + SC::LV_IM + i) : 0u; cii[k] = in ? __ldg(lv + SC::LV_II + i) : 0u; cfr[k] = in ? __ldg(lv + SC::LV_FR + i) : 0u;
        cre[k] = in ? __ldg(lv + SC::LV_RE + i) : 0u; cfl[k] = in ? __ldg(lv + SC::LV_FLAGS + i) : 0u;
    }
#pragma unroll
    for (int k = 0; k < KL; ++k) { const int i = lane + k * G; lvc[k] = (i < SC::LVC_WORDS) ? __ldg(lv + SC::LV_ELEN + i) : 0u; }
#pragma unroll
    for (int k = 0; k < KC; ++k) { const int i = lane + k * G; rad[k] = (i < SC::C) ? __ldg(lv + SC::LV_RAD + i) : 0u; }
#pragma unroll
    for (int k = 0; k < KM; ++k) { const int i = lane + k * G; msk[k] = (i < SC::MASKW) ? __ldg(lv + SC::LV_MASK + i) : 0u; }
    const uint32_t gb = __ldg(lv + SC::LV_GB);
    const uint32_t jab = (SC::J > 0 && lane < SC::J) ? __ldg(lv + SC::LV_JOINT + kJointLevelWords * lane) : 0u;
#pragma unroll
    for (int k = 0; k < KN; ++k) {
        const int i = lane + k * G;
        if (i < SC::N) { smu[SC::BIM + i] = cim[k]; smu[SC::BII + i] = cii[k]; smu[SC::BFR + i] = cfr[k]; smu[SC::BRE + i] = cre[k]; smu[SC::BFL + i] = cfl[k]; }
    }
#pragma unroll
    for (int k = 0; k < KL; ++k) { const int i = lane + k * G; if (i < SC::LVC_WORDS) smu[SC::LVC + i] = lvc[k]; }
#pragma unroll
    for (int k = 0; k < KC; ++k) { const int i = lane + k * G; if (i < SC::C) smu[SC::RAD + i] = rad[k]; }
#pragma unroll
    for (int k = 0; k < KM; ++k) { const int i = lane + k * G; if (i < SC::MASKW) smu[SC::MASK + i] = msk[k]; }
    if (lane == 0) smu[SC::META + META_GB] = gb;
    return jab;
}

// Auto-reset of a finished env: next level (its own, or drawn from the pool by the hash of seed,
// global env index and episode), pose from the level, no accumulated impulses, counters.  Returns the
// packed word of joint number `lane` of the level the env is on afterwards.
template <class SC, int G>
__device__ __noinline__ uint32_t reset_env(uint32_t *smu, const uint32_t *levels, int n_levels, int auto_reset, unsigned long long seed,
                                           long long env_index, unsigned long long *counters, uint32_t jab) {
    Group<G> g;
    const int lane = g.lane;
    const int episode = (int)smu[SC::META + META_EPISODE] + 1;
    int level = (int)smu[SC::META + META_LEVEL];
    g.sync();
    if (auto_reset == 2) {
        const unsigned long long h = mix64(seed + ((unsigned long long)env_index + 1ULL) * 0x9E3779B97F4A7C15ULL +
                                           (unsigned long long)episode * 0xD1B54A32D192ED03ULL);
        const int nl = (int)(h % (unsigned long long)n_levels);
        if (nl != level) { level = nl; jab = load_level_consts<SC, G>(smu, levels + (size_t)nl * SC::LV_WORDS); }
    }
    const uint32_t *lv = levels + (size_t)level * SC::LV_WORDS;
    for (int i = lane; i < 6 * SC::N; i += G) smu[body_word<SC>(i)] = lv[SC::LV_X + i];
    if (SC::J > 0 && lane < SC::J) { smu[SC::JROW + kJointWords * lane + JR_ACCX] = 0u; smu[SC::JROW + kJointWords * lane + JR_ACCY] = 0u; smu[SC::JROW + kJointWords * lane + JR_ACCR] = 0u; }
    for (int i = lane; i < (SC::NPAIRS + 3) / 4; i += G) smu[SC::WIDX + i] = 0xffffffffu;
    if (lane == 0) {
        smu[SC::META + META_STEP] = 0u; smu[SC::META + META_EPISODE] = (uint32_t)episode; smu[SC::META + META_LEVEL] = (uint32_t)level;
        smu[SC::META + META_STATUS] = 0u; smu[SC::META + META_NWARM] = 0u;
        atomicAdd(counters + 1, 1ULL);
    }
    g.sync();
    return jab;
}

// packed work counters of a group to the global ones (lane 0)
__device__ __noinline__ void flush_counters(unsigned long long *counters, unsigned c_surv, unsigned c_rec, unsigned c_man) {
    const unsigned v[6] = { c_man & 0xffffu, c_man >> 16, c_surv & 0xffffu, c_surv >> 16, c_rec & 0xffffu, c_rec >> 16 };
#pragma unroll 1
    for (int q = 0; q < 6; ++q) if (v[q]) atomicAdd(counters + 2 + q, (unsigned long long)v[q]);
}

// debug trace of one pair's manifolds
__device__ __noinline__ void trace_pair(float *t, int nm, unsigned act, float px0, float py0, float pen0, float px1, float py1, float pen1,
                                        float nx0, float ny0, float nx1, float ny1) {
    t[0] = px0; t[1] = py0; t[2] = nx0; t[3] = ny0; t[4] = pen0; t[5] = (act & 1u) ? 1.0f : 0.0f;
    if (nm > 1) { t[6] = px1; t[7] = py1; t[8] = nx1; t[9] = ny1; t[10] = pen1; t[11] = (act & 2u) ? 1.0f : 0.0f; }
}
template <class SC, int G>
__device__ __noinline__ void trace_clear(float *trace) {
    const Group<G> g;
    for (int i = g.lane; i < SC::NSLOTS * 6; i += G) trace[i] = ((i % 6) == 3) ? 1.0f : ((i % 6) == 4 ? -1.0f : 0.0f);
    g.sync();
}

// ---- symbolic per-entity observation of the scene as it stands (paper, tables "Information provided for shapes /
// joints / thrusters"), written after the state record has gone back to memory: the image is built in the part of the
// scene's shared-memory region that only holds per-step data (from the world-frame vertices up) and copied out with
// 16-byte stores.  The same rows, value for value, as k2d_obs_kernel writes.
struct ObsDims { int n_polygons, n_circles, n_joints, n_thrusters, n_actions; };
template <class SC, int G>
__device__ __noinline__ void write_obs(float *sm, const uint32_t *levels, float *obs, ObsDims dims, int e) {
    const Group<G> g;
    const int lane = g.lane;
    const uint32_t *smu = reinterpret_cast<const uint32_t *>(sm);
    const uint32_t *lv = levels + (size_t)smu[SC::META + META_LEVEL] * SC::LV_WORDS;
    const float *lvf = reinterpret_cast<const float *>(lv);
    const int n_shapes = dims.n_polygons + dims.n_circles;
    const int jw = 11 + dims.n_actions;
    const int width = n_shapes * 29 + 2 * dims.n_joints * jw + 6 * dims.n_thrusters;
    float *img = sm + SC::WVX;
    if (ck_idx<CK_OBS>(SC::WVX + width, region_words<SC, G>() + 1) == 0) return;      // cannot be 0 otherwise: the image starts beyond the body arrays
    g.sync();
    for (int i = lane; i < SC::N; i += G) {
        float c, sn;
        sincos_spec(sm[SC::BPOS + 4 * i + 2], c, sn);
        sm[SC::BC + i] = c; sm[SC::BS + i] = sn;
    }
    g.sync();
    for (int ci = lane; ci < n_shapes; ci += G) {
        const int i = ci < dims.n_polygons ? ci : SC::P + (ci - dims.n_polygons);     // internal shape index
        float *o = img + ci * 29;
        const uint32_t fl = smu[SC::BFL + i];
        if (!(fl & F_ACTIVE)) {
            for (int f = 0; f < 29; ++f) o[f] = 0.0f;
            continue;
        }
        const int nv = flag_nverts(fl);
        const uint32_t role = flag_role(fl);
        const bool poly = i < SC::P;
        const float4 p4 = ld4(sm + SC::BPOS + 4 * i), v4 = ld4(sm + SC::BVEL + 4 * i);
        o[0] = p4.x; o[1] = p4.y; o[2] = v4.x; o[3] = v4.y;
        o[4] = sm[SC::BIM + i]; o[5] = sm[SC::BII + i]; o[6] = lvf[SC::LV_DENS + i];
        o[7] = tanh_spec(v4.z * 0.1f);
#pragma unroll
        for (int r = 0; r < 4; ++r) o[8 + r] = (role == (uint32_t)r) ? 1.0f : 0.0f;
        o[12] = sm[SC::BS + i]; o[13] = sm[SC::BC + i]; o[14] = sm[SC::BFR + i]; o[15] = sm[SC::BRE + i];
        o[16] = poly ? 1.0f : 0.0f; o[17] = poly ? 0.0f : 1.0f;
        o[18] = poly ? 0.0f : sm[SC::RAD + (poly ? 0 : i - SC::P)];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool on = poly && k < nv;
            o[19 + 2 * k] = on ? lvf[SC::LV_PVX + 4 * (poly ? i : 0) + k] : 0.0f;
            o[20 + 2 * k] = on ? lvf[SC::LV_PVY + 4 * (poly ? i : 0) + k] : 0.0f;
        }
        o[27] = (poly && nv == 3) ? 1.0f : 0.0f;
        o[28] = (poly && nv != 3) ? 1.0f : 0.0f;
    }
    float *jrows = img + n_shapes * 29;
    for (int row = lane; row < 2 * dims.n_joints; row += G) {
        const int j = row >> 1, d = row & 1;
        const uint32_t *jl = lv + SC::LV_JOINT + kJointLevelWords * j;
        const uint32_t jw0 = jl[0];
        float *o = jrows + row * jw;
        for (int f = 0; f < jw; ++f) o[f] = 0.0f;
        if ((jw0 >> 28) & 1u) {
            const int a = jw0 & 255, b = (jw0 >> 8) & 255;
            const int from = d ? b : a, to = d ? a : b;
            o[0] = 1.0f; o[1] = (jl[10] & 1u) ? 1.0f : 0.0f;
#pragma unroll
            for (int f = 2; f < 6; ++f) { const int side = ((f - 2) >> 1) ^ d; o[f] = __uint_as_float(jl[1 + 2 * side + ((f - 2) & 1)]); }
            o[6] = __uint_as_float(jl[6]); o[7] = __uint_as_float(jl[5]);
            const int bind = (int)((jw0 >> 16) & 255);
            if (bind < dims.n_actions) o[9 + bind] = 1.0f;
            o[9 + dims.n_actions] = __fmaf_rn(sm[SC::BS + to], sm[SC::BC + from], -(sm[SC::BC + to] * sm[SC::BS + from]));
            o[10 + dims.n_actions] = __fmaf_rn(sm[SC::BC + to], sm[SC::BC + from], sm[SC::BS + to] * sm[SC::BS + from]);
        }
    }
    float *trows = jrows + 2 * dims.n_joints * jw;
    for (int t = lane; t < dims.n_thrusters; t += G) {
        const uint32_t *th = lv + SC::LV_THR + 8 * t;
        const uint32_t tp = th[0];
        float *o = trows + t * 6;
        for (int f = 0; f < 6; ++f) o[f] = 0.0f;
        if ((tp >> 20) & 1u) {
            const int i = tp & 255;
            float dx, dy;
            rot2(sm[SC::BC + i], sm[SC::BS + i], __uint_as_float(th[3]), __uint_as_float(th[4]), dx, dy);
            o[0] = 1.0f; o[1] = __uint_as_float(th[1]); o[2] = __uint_as_float(th[2]); o[3] = __uint_as_float(th[5]);
            o[4] = dy; o[5] = dx;
        }
    }
    g.sync();
    float *out = obs + (size_t)e * width;
    if (((width & 3) == 0) && ((reinterpret_cast<uintptr_t>(obs) & 15) == 0)) {
        const float4 *src = reinterpret_cast<const float4 *>(img);
        float4 *dst = reinterpret_cast<float4 *>(out);
        for (int q = lane; q < width / 4; q += G) dst[q] = src[q];
    } else {
        for (int q = lane; q < width; q += G) out[q] = img[q];
    }
    g.sync();
}

// ---------------------------------------------------------------- scene processing
template <class SC, int G>
struct Scene {
    static_assert(SC::J <= G && SC::T <= G && kMaxActions <= 2 * G, "one lane per joint / thruster");
    static_assert(2 * G <= 5 * SC::P4, "positional corrections reuse the world-frame vertex arrays");
    float *sm;            // this scene's shared-memory region
    uint32_t *smu;
    const uint16_t *ptab; // block-shared pair table
    uint32_t *ovf;        // this group's overflow scratch in global memory
    const StepParams &prm;
    Group<G> g;
    int lane;
    // state a lane keeps in registers from step to step
    Rec rec;              // contact pair record number `lane` of the latest step (its accumulated impulses warm-start the next)
    uint32_t jab;         // packed word of joint number `lane` (0 beyond the last joint)
    unsigned c_surv, c_rec, c_man;   // packed work counters: pp | pc << 16, cc | active pairs << 16, manifolds | env-steps << 16

    __device__ __forceinline__ Scene(uint32_t *region, const uint16_t *pt, uint32_t *scratch, const StepParams &p)
        : sm(reinterpret_cast<float *>(region)), smu(region), ptab(pt), ovf(scratch), prm(p), g() {
        lane = g.lane; jab = 0u; c_surv = 0u; c_rec = 0u; c_man = 0u;
    }

    __device__ __forceinline__ uint8_t *surv() { return reinterpret_cast<uint8_t *>(smu + SC::SURV); }
    __device__ __forceinline__ uint8_t *widx() { return reinterpret_cast<uint8_t *>(smu + SC::WIDX); }
    __device__ __forceinline__ float4 &box4(int i) { return *reinterpret_cast<float4 *>(sm + SC::BOX + 4 * i); }
    // this lane's word of per-lane field f
    __device__ __forceinline__ float &lanef(int f) { return sm[SC::STG + f * G + lane]; }
    // this lane's word of field f of its second record (lanes below G / 2 only)
    __device__ __forceinline__ float &ovl(int f) { return sm[SC::STG + LF_COUNT * G + f * (G / 2) + lane]; }
    __device__ __forceinline__ ContactConsts contact_consts() const {
        ContactConsts cc; cc.slop = prm.slop; cc.rest_thr = prm.rest_thr; cc.alpha = prm.contact_alpha; cc.beta = prm.contact_beta; return cc;
    }
    // paper, "Reward": d_t of the dense signal kappa (d_t - d_{t+1})
    __device__ __forceinline__ float green_blue_distance() const {
        const uint32_t gb = smu[SC::META + META_GB];
        const float4 pg = ld4(sm + SC::BPOS + 4 * (gb & 255u)), pb = ld4(sm + SC::BPOS + 4 * ((gb >> 8) & 255u));
        const float dx = pb.x - pg.x, dy = pb.y - pg.y;
        return sqrtf(dot2(dx, dy, dx, dy));
    }
    __device__ __forceinline__ void flush() {
        if (lane == 0) flush_counters(prm.counters, c_surv, c_rec, c_man);
        c_surv = 0u; c_rec = 0u; c_man = 0u;
    }

    // ---- narrowphase: polygon a against polygon b (world data in shared memory)
    __device__ unsigned manifold_pp(int a, int b, Manifold (&m)[2]) const {
        const int cnta = flag_nverts(smu[SC::BFL + a]), cntb = flag_nverts(smu[SC::BFL + b]);
        // largest separation of the other polygon's vertices along each polygon's face normals, first face on ties
        float sa = 0.0f, sb = 0.0f; int ea = 0, eb = 0;
#pragma unroll 1
        for (int side = 0; side < 2; ++side) {
            const int x = side ? b : a, y = side ? a : b;
            const int cntx = side ? cntb : cnta, cnty = side ? cnta : cntb;
            const float4 nx4 = ld4(sm + SC::WNX + 4 * x), ny4 = ld4(sm + SC::WNY + 4 * x), off4 = ld4(sm + SC::WOFF + 4 * x);
            const float4 yx4 = ld4(sm + SC::WVX + 4 * y), yy4 = ld4(sm + SC::WVY + 4 * y);
            const float nxs[4] = { nx4.x, nx4.y, nx4.z, nx4.w }, nys[4] = { ny4.x, ny4.y, ny4.z, ny4.w };
            const float offs[4] = { off4.x, off4.y, off4.z, off4.w };
            const float yx[4] = { yx4.x, yx4.y, yx4.z, yx4.w }, yy[4] = { yy4.x, yy4.y, yy4.z, yy4.w };
            float best = 0.0f; int edge = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (i < cntx) {
                    float lo = dot2(nxs[i], nys[i], yx[0], yy[0]);
#pragma unroll
                    for (int j = 1; j < 4; ++j)
                        if (j < cnty) lo = fmin_cmp(lo, dot2(nxs[i], nys[i], yx[j], yy[j]));
                    const float sep = lo - offs[i];
                    if (i == 0 || sep > best) { best = sep; edge = i; }
                }
            }
            if (side == 0) { sa = best; ea = edge; } else { sb = best; eb = edge; }
        }
        if (sa > 0.0f || sb > 0.0f) return 0u;
        const bool ref_b = sb > sa + prm.face_tol;
        const int R = ref_b ? b : a, I = ref_b ? a : b;
        const int cntr = ref_b ? cntb : cnta, cnti = ref_b ? cnta : cntb;
        const int e = ref_b ? eb : ea;
        const float nx = sm[SC::WNX + 4 * R + e], ny = sm[SC::WNY + 4 * R + e];
        const int e2 = (e + 1 == cntr) ? 0 : e + 1;
        const float v1x = sm[SC::WVX + 4 * R + e], v1y = sm[SC::WVY + 4 * R + e];
        const float v2x = sm[SC::WVX + 4 * R + e2], v2y = sm[SC::WVY + 4 * R + e2];
        int f = 0;
        float fd = dot2(sm[SC::WNX + 4 * I], sm[SC::WNY + 4 * I], nx, ny);
#pragma unroll
        for (int k = 1; k < 4; ++k) {
            if (k < cnti) {
                float d = dot2(sm[SC::WNX + 4 * I + k], sm[SC::WNY + 4 * I + k], nx, ny);
                if (d < fd) { fd = d; f = k; }
            }
        }
        const int f2 = (f + 1 == cnti) ? 0 : f + 1;
        float ipx[2] = { sm[SC::WVX + 4 * I + f], sm[SC::WVX + 4 * I + f2] };
        float ipy[2] = { sm[SC::WVY + 4 * I + f], sm[SC::WVY + 4 * I + f2] };
        const float tx = -ny, ty = nx;
        const float lo = dot2(tx, ty, v1x, v1y), hi = dot2(tx, ty, v2x, v2y);
        const float s0 = dot2(tx, ty, ipx[0], ipy[0]), s1 = dot2(tx, ty, ipx[1], ipy[1]);
        if ((s0 < lo && s1 < lo) || (s0 > hi && s1 > hi)) return 0u;
        float cx[2] = { ipx[0], ipx[1] }, cy[2] = { ipy[0], ipy[1] };
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const float sk = k ? s1 : s0, so = k ? s0 : s1;
            bool clip = false; float bound = lo;
            if (sk < lo) { bound = lo; clip = true; }
            else if (sk > hi) { bound = hi; clip = true; }
            if (clip) {
                float t = (bound - sk) / (so - sk);
                cx[k] = __fmaf_rn(t, ipx[1 - k] - ipx[k], ipx[k]);
                cy[k] = __fmaf_rn(t, ipy[1 - k] - ipy[k], ipy[k]);
            }
        }
        const float off = sm[SC::WOFF + 4 * R + e];
        unsigned act = 0u;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            m[k].pen = off - dot2(nx, ny, cx[k], cy[k]);
            m[k].px = cx[k]; m[k].py = cy[k];
            m[k].nx = ref_b ? -nx : nx; m[k].ny = ref_b ? -ny : ny;
            if (m[k].pen > 0.0f) act |= 1u << k;
        }
        return act;
    }

    // polygon a against circle b
    __device__ unsigned manifold_pc(int a, int b, Manifold &m) const {
        const int cnt = flag_nverts(smu[SC::BFL + a]);
        const float cx = sm[SC::BPOS + 4 * b], cy = sm[SC::BPOS + 4 * b + 1], r = sm[SC::RAD + (b - SC::P)];
        float maxsep = 0.0f, mind2 = 0.0f, qx = 0.0f, qy = 0.0f, dqx = 0.0f, dqy = 0.0f;
        int kmax = 0, kmin = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (k < cnt) {
                const float nx = sm[SC::WNX + 4 * a + k], ny = sm[SC::WNY + 4 * a + k];
                const float wx = sm[SC::WVX + 4 * a + k], wy = sm[SC::WVY + 4 * a + k];
                const float sep = dot2(nx, ny, cx, cy) - sm[SC::WOFF + 4 * a + k];
                const float tx = -ny, ty = nx;
                float s = dot2(tx, ty, cx - wx, cy - wy);
                s = fmax_cmp(fmin_cmp(s, sm[SC::LVC + 4 * a + k]), 0.0f);
                const float px = __fmaf_rn(s, tx, wx), py = __fmaf_rn(s, ty, wy);
                const float ex = cx - px, ey = cy - py;
                const float d2 = dot2(ex, ey, ex, ey);
                if (k == 0 || sep > maxsep) { maxsep = sep; kmax = k; }
                if (k == 0 || d2 < mind2) { mind2 = d2; kmin = k; qx = px; qy = py; dqx = ex; dqy = ey; }
            }
        }
        if (maxsep > 0.0f) {
            const float d = sqrtf(mind2);
            if (d < 1e-9f) { m.nx = sm[SC::WNX + 4 * a + kmin]; m.ny = sm[SC::WNY + 4 * a + kmin]; }
            else { const float inv = 1.0f / d; m.nx = dqx * inv; m.ny = dqy * inv; }
            m.pen = r - d; m.px = qx; m.py = qy;
        } else {
            m.nx = sm[SC::WNX + 4 * a + kmax]; m.ny = sm[SC::WNY + 4 * a + kmax];
            m.pen = r - maxsep;
            m.px = __fmaf_rn(-maxsep, m.nx, cx); m.py = __fmaf_rn(-maxsep, m.ny, cy);
        }
        return m.pen > 0.0f ? 1u : 0u;
    }

    __device__ unsigned manifold_cc(int a, int b, Manifold &m) const {
        const float ax = sm[SC::BPOS + 4 * a], ay = sm[SC::BPOS + 4 * a + 1], ra = sm[SC::RAD + (a - SC::P)];
        const float dx = sm[SC::BPOS + 4 * b] - ax, dy = sm[SC::BPOS + 4 * b + 1] - ay, rb = sm[SC::RAD + (b - SC::P)];
        const float dist = sqrtf(dot2(dx, dy, dx, dy));
        if (dist < 1e-9f) { m.nx = 0.0f; m.ny = 1.0f; }
        else { const float inv = 1.0f / dist; m.nx = dx * inv; m.ny = dy * inv; }
        m.pen = (ra + rb) - dist;
        m.px = __fmaf_rn(ra, m.nx, ax); m.py = __fmaf_rn(ra, m.ny, ay);
        return m.pen > 0.0f ? 1u : 0u;
    }

    // ---- one visit of this lane's contact pair record.  MODE 0: warm start, 1: solver iteration, 2: positional correction
    template <int MODE>
    __device__ __forceinline__ void visit_pair() {
        const uint32_t ab = rec.ab;
        const int a = ck_idx<CK_BODY>(ab & 31, SC::N), b = ck_idx<CK_BODY>((ab >> 5) & 31, SC::N);
        const unsigned amask = (ab >> 10) & 3u;
        const bool dyn_a = (ab >> 26) & 1u, dyn_b = (ab >> 27) & 1u;
        if (MODE == 2) {
            correct_pair(sm + SC::BPOS, a, b, amask, dyn_a, dyn_b, rec.nx, rec.ny, rec.ma, rec.mb,
                         sm[SC::WVX + lane], sm[SC::WVX + G + lane]);
            return;
        }
        const float4 va4 = ld4(sm + SC::BVEL + 4 * a), vb4 = ld4(sm + SC::BVEL + 4 * b);
        float vax = va4.x, vay = va4.y, wa = va4.z, vbx = vb4.x, vby = vb4.y, wb = vb4.z;
        if (amask & 1u)
            manifold_rows<MODE>(rec.nx, rec.ny, rec.mu, rec.ma, rec.mb, rec.ia, rec.ib, rec.rna, rec.rnb, rec.rta, rec.rtb,
                                rec.massn, rec.masst, rec.target, rec.accn, rec.acct, vax, vay, wa, vbx, vby, wb);
        if (amask & 2u) {
            float accn = lanef(LF_ACC2N), acct = lanef(LF_ACC2T);
            manifold_rows<MODE>(rec.nx, rec.ny, rec.mu, rec.ma, rec.mb, rec.ia, rec.ib, lanef(M2_RNA), lanef(M2_RNB), lanef(M2_RTA),
                                lanef(M2_RTB), lanef(M2_MASSN), lanef(M2_MASST), lanef(M2_TARGET), accn, acct, vax, vay, wa, vbx, vby, wb);
            if (MODE == 1) { lanef(LF_ACC2N) = accn; lanef(LF_ACC2T) = acct; }
        }
        if (dyn_a) st4(sm + SC::BVEL + 4 * a, vax, vay, wa);
        if (dyn_b) st4(sm + SC::BVEL + 4 * b, vbx, vby, wb);
    }
    // records of one level touch disjoint movable bodies; levels in order keep the record order
    template <int MODE>
    __device__ __forceinline__ void sweep_pairs(int cmax, int clevel, int clevel2) {
#pragma unroll 1
        for (int lvl = 1; lvl <= cmax; ++lvl) {
            if (clevel == lvl) visit_pair<MODE>();
            if (clevel2 == lvl) visit_second<SC, G, MODE>(sm);
            g.sync();
        }
    }

    // ---- one environment step
    __device__ __forceinline__ void step(int e, int s) {
        // frozen env: reports done, nothing else
        if (smu[SC::META + META_STATUS] & 1u) {
            if (lane == 0) { prm.reward[(size_t)s * prm.n_envs + e] = 0.0f; prm.done[(size_t)s * prm.n_envs + e] = 1; }
            return;
        }
        K2D_PHASE_BEGIN();
        const uint32_t *lv = prm.levels + (size_t)ck_idx<CK_LEVEL_ID>((int)smu[SC::META + META_LEVEL], prm.n_levels) * SC::LV_WORDS;
        // dense reward: distance between the first green and the first blue shape before the step
        if (prm.dense_kappa != 0.0f && lane == 0) sm[SC::META + META_D0] = green_blue_distance();
        // actions of this step
        const float *act_row = prm.actions + ((size_t)(s / prm.frame_skip) * prm.n_envs + e) * prm.n_actions;
        if (lane < prm.n_actions) sm[SC::ACT + lane] = act_row[lane];
        if (G < kMaxActions && lane + G < prm.n_actions) sm[SC::ACT + lane + G] = act_row[lane + G];
        // the body-frame vertices and normals this lane will turn are asked for now and used after the rotations are known
        constexpr int KV = (SC::P4 + G - 1) / G;
        float pvx[KV], pvy[KV], pnx[KV], pny[KV];
#pragma unroll
        for (int k = 0; k < KV; ++k) {
            const int v = lane + k * G; const bool in = v < SC::P4;
            pvx[k] = in ? __uint_as_float(__ldg(lv + SC::LV_PVX + v)) : 0.0f; pvy[k] = in ? __uint_as_float(__ldg(lv + SC::LV_PVY + v)) : 0.0f;
            pnx[k] = in ? __uint_as_float(__ldg(lv + SC::LV_PNX + v)) : 0.0f; pny[k] = in ? __uint_as_float(__ldg(lv + SC::LV_PNY + v)) : 0.0f;
        }
        // gravity, rotation, circle boxes
        for (int i = lane; i < SC::N; i += G) {
            const uint32_t fl = smu[SC::BFL + i];
            if ((fl & F_ACTIVE) && (fl & F_DYNAMIC)) sm[SC::BVEL + 4 * i + 1] = sm[SC::BVEL + 4 * i + 1] + prm.gdt;
            float c, sn;
            sincos_spec(sm[SC::BPOS + 4 * i + 2], c, sn);
            sm[SC::BC + i] = c; sm[SC::BS + i] = sn;
            if (i >= SC::P) {
                const float r = sm[SC::RAD + (i - SC::P)], x = sm[SC::BPOS + 4 * i], y = sm[SC::BPOS + 4 * i + 1];
                box4(i) = make_float4(x - r, y - r, x + r, y + r);
            }
        }
        g.sync();
        // world-frame polygon vertices, normals, face offsets
#pragma unroll
        for (int kk = 0; kk < KV; ++kk) {
            const int v = lane + kk * G;
            const int i = v >> 2, k = v & 3;
            if (v < SC::P4 && k < (int)flag_nverts(smu[SC::BFL + i])) {
                const float c = sm[SC::BC + i], sn = sm[SC::BS + i];
                float rx, ry, nx, ny;
                rot2(c, sn, pvx[kk], pvy[kk], rx, ry);
                rot2(c, sn, pnx[kk], pny[kk], nx, ny);
                const float wx = rx + sm[SC::BPOS + 4 * i], wy = ry + sm[SC::BPOS + 4 * i + 1];
                sm[SC::WVX + v] = wx; sm[SC::WVY + v] = wy; sm[SC::WNX + v] = nx; sm[SC::WNY + v] = ny;
                sm[SC::WOFF + v] = dot2(nx, ny, wx, wy);
            }
        }
        // this lane's joint: "on" bit and level come with the level record
        const int jlevel = ((jab >> 24) & 1u) ? (int)((jab >> 25) & 7u) : 0;
        const int jmax = (SC::J > 0) ? g.max_int(jlevel) : 0;
        g.sync();
        // polygon boxes
        for (int i = lane; i < SC::P; i += G) {
            const int cntv = flag_nverts(smu[SC::BFL + i]);
            float x0 = sm[SC::WVX + 4 * i], y0 = sm[SC::WVY + 4 * i], x1 = x0, y1 = y0;
#pragma unroll
            for (int k = 1; k < 4; ++k) {
                if (k < cntv) {
                    const float x = sm[SC::WVX + 4 * i + k], y = sm[SC::WVY + 4 * i + k];
                    x0 = fmin_cmp(x0, x); y0 = fmin_cmp(y0, y); x1 = fmax_cmp(x1, x); y1 = fmax_cmp(y1, y);
                }
            }
            box4(i) = make_float4(x0, y0, x1, y1);
        }
        K2D_PHASE(PH_GEOMETRY);
        // motors (joint order), thrusters (thruster order)
        sweep_joints<SC, G, 3>(sm, jab, lane, jlevel, jmax, prm.motor_rho, prm.discrete);
        if (SC::T > 0) {
            int tl = 0; uint32_t tp = 0u;
            const uint32_t *th = smu + SC::LVC + (SC::LV_THR - SC::LV_ELEN) + 8 * lane;
            if (lane < SC::T) { tp = th[0]; if ((tp >> 16) & 1u) tl = (tp >> 17) & 7u; }
            const int tmax = g.max_int(tl);
#pragma unroll 1
            for (int lvl = 1; lvl <= tmax; ++lvl) {
                if (tl == lvl) {
                    const int i = ck_idx<CK_BODY>(tp & 255, SC::N);
                    const float tv = sm[SC::ACT + ck_idx<CK_COUNT>((tp >> 8) & 255, kMaxActions)];
                    // continuous in [0, 1], or multi-discrete: 0 off, anything else full power
                    const float A = prm.discrete ? (__float_as_int(tv) != 0 ? 1.0f : 0.0f) : fmax_cmp(fmin_cmp(tv, 1.0f), 0.0f);
                    const float c = sm[SC::BC + i], sn = sm[SC::BS + i];
                    float dx, dy, rx, ry;
                    rot2(c, sn, __uint_as_float(th[3]), __uint_as_float(th[4]), dx, dy);
                    rot2(c, sn, __uint_as_float(th[1]), __uint_as_float(th[2]), rx, ry);
                    const float imp = (__uint_as_float(th[5]) * A) * prm.dt;
                    const float jx = imp * dx, jy = imp * dy;
                    const float im = sm[SC::BIM + i];
                    sm[SC::BVEL + 4 * i] = __fmaf_rn(jx, im, sm[SC::BVEL + 4 * i]);
                    sm[SC::BVEL + 4 * i + 1] = __fmaf_rn(jy, im, sm[SC::BVEL + 4 * i + 1]);
                    sm[SC::BVEL + 4 * i + 2] = __fmaf_rn(cross2(rx, ry, jx, jy), sm[SC::BII + i], sm[SC::BVEL + 4 * i + 2]);
                }
                g.sync();
            }
        }
        K2D_PHASE(PH_ACTUATORS);
        // joint pre-step (poses only; velocities are not read): the row goes to shared memory
        if (SC::J > 0 && lane < SC::J) {
            float *jr = sm + SC::JROW + kJointWords * lane;
            if (!((jab >> 24) & 1u) || !prm.warm_start) { jr[JR_ACCX] = 0.0f; jr[JR_ACCY] = 0.0f; jr[JR_ACCR] = 0.0f; }
            int ang = 0;
            float kr = 0.0f, bias_r = 0.0f;
            if ((jab >> 24) & 1u) {
                const int a = ck_idx<CK_BODY>(jab & 255, SC::N), b = ck_idx<CK_BODY>((jab >> 8) & 255, SC::N);
                const uint32_t *jl = smu + SC::LVC + (SC::LV_JOINT - SC::LV_ELEN) + kJointLevelWords * lane;
                float rax, ray, rbx, rby;
                rot2(sm[SC::BC + a], sm[SC::BS + a], __uint_as_float(jl[1]), __uint_as_float(jl[2]), rax, ray);
                rot2(sm[SC::BC + b], sm[SC::BS + b], __uint_as_float(jl[3]), __uint_as_float(jl[4]), rbx, rby);
                const float ma = sm[SC::BIM + a], mb = sm[SC::BIM + b], ia = sm[SC::BII + a], ib = sm[SC::BII + b];
                jr[JR_MA] = ma; jr[JR_MB] = mb; jr[JR_IA] = ia; jr[JR_IB] = ib;
                const float gx = (sm[SC::BPOS + 4 * b] + rbx) - (sm[SC::BPOS + 4 * a] + rax), gy = (sm[SC::BPOS + 4 * b + 1] + rby) - (sm[SC::BPOS + 4 * a + 1] + ray);
                const float msum = ma + mb;
                float k11 = msum; k11 = __fmaf_rn(ia * ray, ray, k11); k11 = __fmaf_rn(ib * rby, rby, k11);
                float k22 = msum; k22 = __fmaf_rn(ia * rax, rax, k22); k22 = __fmaf_rn(ib * rbx, rbx, k22);
                float k12 = -((ia * rax) * ray); k12 = __fmaf_rn(-(ib * rbx), rby, k12);
                const float det = __fmaf_rn(k11, k22, -(k12 * k12));
                const float inv_det = 1.0f / det;
                jr[JR_RAX] = rax; jr[JR_RAY] = ray; jr[JR_RBX] = rbx; jr[JR_RBY] = rby;
                jr[JR_I11] = k22 * inv_det; jr[JR_I22] = k11 * inv_det; jr[JR_I12] = -(k12 * inv_det);
                jr[JR_BX] = prm.joint_alpha * gx; jr[JR_BY] = prm.joint_alpha * gy;
                const float share = prm.joint_beta / msum;
                jr[JR_CX] = share * gx; jr[JR_CY] = share * gy;
                // angular row from the relative rotation at the start of the step
                const float isum = ia + ib;
                const uint32_t kind = jl[10];
                if (isum > 0.0f && kind != 0u) {
                    const float rel = sm[SC::BPOS + 4 * a + 2] - sm[SC::BPOS + 4 * b + 2];
                    if (kind & 1u) { ang = 1; kr = 1.0f / isum; bias_r = prm.joint_gamma * (rel - __uint_as_float(jl[7])); }
                    else {
                        const float lo = __uint_as_float(jl[8]), hi = __uint_as_float(jl[9]);
                        if (rel > hi) { ang = 2; kr = 1.0f / isum; bias_r = prm.joint_gamma * (rel - hi); }
                        else if (rel < lo) { ang = 3; kr = 1.0f / isum; bias_r = prm.joint_gamma * (rel - lo); }
                    }
                }
            }
            if (ang != 1) jr[JR_ACCR] = 0.0f;
            jr[JR_ANG] = __int_as_float(ang); jr[JR_KR] = kr; jr[JR_BIASR] = bias_r;
        }
        g.sync();

        K2D_PHASE(PH_JOINT_PRESTEP);
        // bounding-box test over all pairs -> compact list of surviving pairs, in pair order
        int nsurv = 0, ns_pp, ns_pc;
        {
            int mine_pp = 0, mine_pc = 0;     // this lane's survivors below the polygon-circle / circle-circle boundary
            const float mg = prm.aabb_margin;
#pragma unroll 2
            for (int base = 0; base < SC::NPAIRS; base += G) {
                const int p = base + lane;
                bool keep = false;
                if (p < SC::NPAIRS && ((smu[SC::MASK + (p >> 5)] >> (p & 31)) & 1u)) {
                    const uint32_t code = ptab[p];
                    const float4 ba = box4(code & 255), bb = box4(code >> 8);
                    keep = !(ba.z + mg < bb.x || bb.z + mg < ba.x || ba.w + mg < bb.y || bb.w + mg < ba.y);
                }
                const unsigned bal = g.ballot(keep);
                if (keep) surv()[ck_idx<CK_STAGE>(nsurv + __popc(bal & g.lanes_below()), SC::NPAIRS)] = (uint8_t)p;
                nsurv += __popc(bal);
                mine_pp += (keep && p < SC::NPP) ? 1 : 0;
                mine_pc += (keep && p < SC::NPP + SC::NPC) ? 1 : 0;
            }
            ns_pp = g.sum_int(mine_pp);
            ns_pc = g.sum_int(mine_pc);
        }
        g.sync();
        c_surv += (unsigned)ns_pp | ((unsigned)(ns_pc - ns_pp) << 16);
        c_rec += (unsigned)(nsurv - ns_pc);

        K2D_PHASE(PH_BOX_TEST);
        // narrowphase: survivors of one kind at a time; active pairs are staged in pair order
        int nrec = 0;
        bool t_gb = false, t_gr = false;
        float *trace = prm.trace ? prm.trace + (size_t)e * SC::NSLOTS * 6 : nullptr;
        if (trace) trace_clear<SC, G>(trace);
#pragma unroll 1
        for (int kind = 0; kind < 3; ++kind) {
            const int lo = kind == 0 ? 0 : (kind == 1 ? ns_pp : ns_pc);
            const int hi = kind == 0 ? ns_pp : (kind == 1 ? ns_pc : nsurv);
#pragma unroll 1
            for (int base = lo; base < hi; base += G) {
                const int idx = base + lane;
                unsigned act = 0u;
                Manifold m[2];
                m[1].px = 0.0f; m[1].py = 0.0f; m[1].pen = 0.0f;
                int p = 0, a = 0, b = 0;
                if (idx < hi) {
                    p = ck_idx<CK_PAIR>(surv()[idx], SC::NPAIRS); a = ck_idx<CK_BODY>(ptab[p] & 255, SC::N); b = ck_idx<CK_BODY>(ptab[p] >> 8, SC::N);
                    if (kind == 0) act = manifold_pp(a, b, m);
                    else if (kind == 1) act = manifold_pc(a, b, m[0]);
                    else act = manifold_cc(a, b, m[0]);
                    // a polygon pair rejected before its manifolds exist leaves its slots at the default
                    if (trace && !(kind == 0 && act == 0u))
                        trace_pair(trace + ((p < SC::NPP) ? 2 * p : SC::NPP + p) * 6, (kind == 0) ? 2 : 1, act, m[0].px, m[0].py, m[0].pen,
                                   m[1].px, m[1].py, m[1].pen, m[0].nx, m[0].ny, m[1].nx, m[1].ny);
                }
                const unsigned bal = g.ballot(act != 0u);
                if (act) {
                    const int k = ck_idx<CK_STAGE>(nrec + __popc(bal & g.lanes_below()), SC::NPAIRS);
                    const uint32_t fa = smu[SC::BFL + a], fb = smu[SC::BFL + b];
                    const uint32_t ra = flag_role(fa), rb = flag_role(fb);
                    t_gb |= (ra == 1u && rb == 2u) || (ra == 2u && rb == 1u);
                    t_gr |= (ra == 1u && rb == 3u) || (ra == 3u && rb == 1u);
                    const uint32_t ab = (uint32_t)a | ((uint32_t)b << 5) | (act << 10) | ((uint32_t)p << 12) |
                                        (((fa & F_DYNAMIC) ? 1u : 0u) << 26) | (((fb & F_DYNAMIC) ? 1u : 0u) << 27);
                    const float nx = (act & 1u) ? m[0].nx : m[1].nx, ny = (act & 1u) ? m[0].ny : m[1].ny;
                    if (k < G) {
                        float *st = sm + SC::STG + k;
                        st[S_AB * G] = __uint_as_float(ab); st[S_NX * G] = nx; st[S_NY * G] = ny;
                        st[S_PX0 * G] = m[0].px; st[S_PY0 * G] = m[0].py; st[S_PEN0 * G] = m[0].pen;
                        st[S_PX1 * G] = m[1].px; st[S_PY1 * G] = m[1].py; st[S_PEN1 * G] = m[1].pen;
                    } else if (k < G + G / 2) {
                        float *st = sm + SC::STG + LF_COUNT * G + (k - G);
                        constexpr int H = G / 2;
                        st[ovs(S_AB) * H] = __uint_as_float(ab); st[ovs(S_NX) * H] = nx; st[ovs(S_NY) * H] = ny;
                        st[ovs(S_PX0) * H] = m[0].px; st[ovs(S_PY0) * H] = m[0].py; st[ovs(S_PEN0) * H] = m[0].pen;
                        st[ovs(S_PX1) * H] = m[1].px; st[ovs(S_PY1) * H] = m[1].py; st[ovs(S_PEN1) * H] = m[1].pen;
                    } else {
                        uint32_t *st = ovf + (size_t)ck_idx<CK_RECORD>(k, SC::NPAIRS) * kRecWords;
                        st[S_AB] = ab; st[S_NX] = __float_as_uint(nx); st[S_NY] = __float_as_uint(ny);
                        st[S_PX0] = __float_as_uint(m[0].px); st[S_PY0] = __float_as_uint(m[0].py); st[S_PEN0] = __float_as_uint(m[0].pen);
                        st[S_PX1] = __float_as_uint(m[1].px); st[S_PY1] = __float_as_uint(m[1].py); st[S_PEN1] = __float_as_uint(m[1].pen);
                    }
                }
                nrec += __popc(bal);
            }
        }
        const bool touch_gb = g.any(t_gb), touch_gr = g.any(t_gr);
        g.sync();
        c_rec += (unsigned)nrec << 16;

        K2D_PHASE(PH_NARROWPHASE);
        // Crowded scenes go through the memory records; with the batched contact solve asked for, so does every scene with
        // second records (more touching pairs than lanes).  The others run their batches from the lanes' records, below.
        const bool overflow = nrec > G + G / 2 || (prm.n_batches > 0 && nrec > G);
        int cmax = 0, clevel = 0, clevel2 = 0;
        if (overflow) {
            cmax = slow_solve<SC, G>(sm, ovf, nrec, jab, jlevel, jmax, prm.solver_iters, prm.warm_start, prm.motor_rho,
                                     rec.accn, rec.acct, contact_consts(), prm.n_batches);
            K2D_PHASE(PH_MEMORY_RECORD_SOLVE);
        } else {
            const ContactConsts cc = contact_consts();
            const bool two = nrec > G;      // some lanes get a second record
            if (two) {
                if (lane == 0) cmax = levels_by_one_lane<SC, G>(smu, ovf, nrec);
                g.sync();
            }
            // every staged pair becomes a record in its own lane: accumulated impulses of the same pair in the
            // previous step come from wherever its record was then
            const bool mine = lane < nrec;
            uint32_t ab = 0u;
            float nx = 0.0f, ny = 0.0f, pt[6] = { 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f };
            float w[4];
            {
                int wi = 255;
                if (mine) {
                    ab = __float_as_uint(lanef(S_AB)); wi = widx()[ck_idx<CK_PAIR>((ab >> 12) & 127, SC::NPAIRS)];
                    nx = lanef(S_NX); ny = lanef(S_NY);
                    pt[0] = lanef(S_PX0); pt[1] = lanef(S_PY0); pt[2] = lanef(S_PEN0); pt[3] = lanef(S_PX1); pt[4] = lanef(S_PY1); pt[5] = lanef(S_PEN1);
                }
                const float old_n = rec.accn, old_t = rec.acct;
                warm_lookup<SC, G>(g, sm, ovf, wi, old_n, old_t, prm.warm_start, w);
                if (two) second_lookup<SC, G>(sm, ovf, nrec, old_n, old_t, prm.warm_start);
            }
            g.sync();     // every lane has read the fields it needs from other lanes before they are rewritten
            const int a = ck_idx<CK_BODY>(ab & 31, SC::N), b = ck_idx<CK_BODY>((ab >> 5) & 31, SC::N);
            const unsigned amask = (ab >> 10) & 3u;
            rec.ab = ab; rec.nx = nx; rec.ny = ny;
            rec.ma = sm[SC::BIM + a]; rec.mb = sm[SC::BIM + b]; rec.ia = sm[SC::BII + a]; rec.ib = sm[SC::BII + b];
            {
                const float fra = sm[SC::BFR + a], frb = sm[SC::BFR + b];
                rec.mu = sqrtf(__fmaf_rn(fra, fra, frb * frb));
            }
            const float er = fmin_cmp(sm[SC::BRE + a], sm[SC::BRE + b]);
            float corr0 = 0.0f, corr1 = 0.0f;
            rec.rna = 0.0f; rec.rnb = 0.0f; rec.rta = 0.0f; rec.rtb = 0.0f; rec.massn = 0.0f; rec.masst = 0.0f; rec.target = 0.0f;
            rec.accn = 0.0f; rec.acct = 0.0f;
            if (amask & 1u) {
                prestep_manifold<SC>(a, b, nx, ny, rec.ma, rec.mb, rec.ia, rec.ib, pt[0], pt[1], pt[2], er, sm, cc,
                                     rec.rna, rec.rnb, rec.rta, rec.rtb, rec.massn, rec.masst, rec.target, corr0);
                rec.accn = w[0]; rec.acct = w[1];
            }
            float acc2n = 0.0f, acc2t = 0.0f;
            if (amask & 2u) {
                float rna, rnb, rta, rtb, massn, masst, target;
                prestep_manifold<SC>(a, b, nx, ny, rec.ma, rec.mb, rec.ia, rec.ib, pt[3], pt[4], pt[5], er, sm, cc,
                                     rna, rnb, rta, rtb, massn, masst, target, corr1);
                lanef(M2_RNA) = rna; lanef(M2_RNB) = rnb; lanef(M2_RTA) = rta; lanef(M2_RTB) = rtb;
                lanef(M2_MASSN) = massn; lanef(M2_MASST) = masst; lanef(M2_TARGET) = target;
                acc2n = w[2]; acc2t = w[3];
            }
            lanef(LF_ACC2N) = acc2n; lanef(LF_ACC2T) = acc2t;
            sm[SC::WVX + lane] = corr0; sm[SC::WVX + G + lane] = corr1;
            K2D_PHASE(PH_RECORDS);
            if (two) {
                const unsigned r2 = second_build<SC, G>(sm, nrec, cc);     // level | active manifolds << 8
                clevel2 = (int)(r2 & 127u);
                clevel = (int)((ab >> 19) & 127u);
                cmax = g.shfl(cmax, 0);
                c_man += (unsigned)g.sum_int((int)(r2 >> 8));
            } else {
                // levels of the records (canonical order = record order): one more than the highest level of an
                // earlier record that shares a movable body.  Every movable body collects the set of records that
                // touch it; a record's conflicts are the earlier members of its bodies' sets; then level r goes to
                // the records whose conflicts all have a level already, round after round.
                uint32_t *touch = smu + SC::SURV;            // the survivor list is no longer needed
                for (int i = lane; i < SC::N; i += G) touch[i] = 0u;
                g.sync();
                const bool da = (ab >> 26) & 1u, db = (ab >> 27) & 1u;
                if (mine && da) atomicOr(touch + a, 1u << lane);
                if (mine && db) atomicOr(touch + b, 1u << lane);
                g.sync();
                const unsigned conflicts = ((da ? touch[a] : 0u) | (db ? touch[b] : 0u)) & g.lanes_below();
                const unsigned all = g.ballot(mine);
                unsigned assigned = 0u;
                int lvl = 0;
#pragma unroll 1
                for (int r = 1; assigned != all; ++r) {
                    const bool ready = mine && lvl == 0 && (conflicts & ~assigned) == 0u;
                    if (ready) lvl = r;
                    assigned |= g.ballot(ready);
                }
                clevel = lvl;
                cmax = g.max_int(lvl);
            }
            K2D_PHASE(PH_LEVELS);
            const int nman = __popc(g.ballot(amask & 1u)) + __popc(g.ballot(amask & 2u));
            c_man += (unsigned)nman;
            // The i-th active manifold goes to batch i mod n_batches: with no more active manifolds than batches every batch
            // holds at most one row and the batched order is the sequential one, which the level schedule reproduces.
            const bool batched = prm.n_batches > 0 && nman > prm.n_batches;
            // warm start: contacts, then joints
            sweep_pairs<0>(cmax, clevel, clevel2);
            sweep_joints<SC, G, 0>(sm, jab, lane, jlevel, jmax, prm.motor_rho);
            K2D_PHASE(PH_WARM_START);
            // solver iterations: joints, then contacts
            if (batched) {
                const float2 acc = batched_iterations<SC, G>(sm, rec, jab, jlevel, jmax, cmax, clevel, prm.solver_iters, prm.motor_rho, prm.n_batches);
                rec.accn = acc.x; rec.acct = acc.y;
            } else {
#pragma unroll 1
                for (int it = 0; it < prm.solver_iters; ++it) {
                    sweep_joints<SC, G, 1>(sm, jab, lane, jlevel, jmax, prm.motor_rho);
                    sweep_pairs<1>(cmax, clevel, clevel2);
                }
            }
        }
        if (!overflow) K2D_PHASE(PH_ITERATIONS);
        // Euler step with the solved velocities
        for (int i = lane; i < SC::N; i += G) {
            if (smu[SC::BFL + i] & F_ACTIVE) {
                const float4 p4 = ld4(sm + SC::BPOS + 4 * i), v4 = ld4(sm + SC::BVEL + 4 * i);
                st4(sm + SC::BPOS + 4 * i, __fmaf_rn(prm.dt, v4.x, p4.x), __fmaf_rn(prm.dt, v4.y, p4.y), __fmaf_rn(prm.dt, v4.z, p4.z));
            }
        }
        g.sync();
        if (overflow) slow_correct<SC, G>(sm, ovf, nrec, cmax);
        else sweep_pairs<2>(cmax, clevel, clevel2);
        sweep_joints<SC, G, 2>(sm, jab, lane, jlevel, jmax, prm.motor_rho);
        bool finite = true;
        for (int i = lane; i < SC::N; i += G) {
            const float4 p4 = ld4(sm + SC::BPOS + 4 * i), v4 = ld4(sm + SC::BVEL + 4 * i);
            finite = finite && finite_bits(p4.x) && finite_bits(p4.y) && finite_bits(p4.z) && finite_bits(v4.x) && finite_bits(v4.y) && finite_bits(v4.z);
        }
        finite = !g.any(!finite);

        K2D_PHASE(PH_INTEGRATE_CORRECT);
        // where the pairs of this step keep their accumulated impulses for the next one
        for (int i = lane; i < (SC::NPAIRS + 3) / 4; i += G) smu[SC::WIDX + i] = 0xffffffffu;
        const int step_count = (int)smu[SC::META + META_STEP] + 1;
        g.sync();
        if (overflow) {
            c_man += (unsigned)slow_finish<SC, G>(sm, ovf, nrec);
            // the first G + G / 2 pairs go back to their lanes
            const uint32_t *wr = ovf + SC::SCRATCH_WARM + (size_t)lane * kWarmWords, *wr2 = wr + (size_t)G * kWarmWords;
            rec.ab = 0u; rec.accn = 0.0f; rec.acct = 0.0f;
            lanef(LF_ACC2N) = 0.0f; lanef(LF_ACC2T) = 0.0f;
            if (lane < nrec) {
                rec.ab = wr[0] << 12;
                rec.accn = __uint_as_float(wr[1]); rec.acct = __uint_as_float(wr[2]);
                lanef(LF_ACC2N) = __uint_as_float(wr[3]); lanef(LF_ACC2T) = __uint_as_float(wr[4]);
            }
            if (lane < G / 2 && G + lane < nrec) {
                ovl(R_AB) = __uint_as_float(wr2[0] << 12);
                ovl(OV_ACC0N) = __uint_as_float(wr2[1]); ovl(OV_ACC0T) = __uint_as_float(wr2[2]);
                ovl(OV_ACC1N) = __uint_as_float(wr2[3]); ovl(OV_ACC1T) = __uint_as_float(wr2[4]);
            }
        } else {
            if (lane < nrec) widx()[ck_idx<CK_PAIR>((rec.ab >> 12) & 127, SC::NPAIRS)] = (uint8_t)lane;
            if (clevel2 != 0) widx()[ck_idx<CK_PAIR>((__float_as_uint(ovl(R_AB)) >> 12) & 127, SC::NPAIRS)] = (uint8_t)(G + lane);
        }

        // reward, termination, counters, auto-reset
        const bool timeout = prm.max_episode_steps > 0 && step_count >= prm.max_episode_steps;
        float reward = (float)((int)touch_gb - (int)touch_gr);
        if (prm.dense_kappa != 0.0f && ((smu[SC::META + META_GB] >> 16) & 1u))
            reward = reward + prm.dense_kappa * (sm[SC::META + META_D0] - green_blue_distance());
        bool done = touch_gb || touch_gr || timeout;
        if (!finite) { reward = 0.0f; done = true; }
        if (lane == 0) {
            prm.reward[(size_t)s * prm.n_envs + e] = reward;
            prm.done[(size_t)s * prm.n_envs + e] = done ? 1 : 0;
            smu[SC::META + META_STEP] = (uint32_t)step_count;
            smu[SC::META + META_NWARM] = (uint32_t)nrec;
            if (!finite) { smu[SC::META + META_STATUS] |= 1u; atomicAdd(prm.counters + 0, 1ULL); }
        }
        c_man += 1u << 16;
        g.sync();
        if (done && prm.auto_reset != 0)
            jab = reset_env<SC, G>(smu, prm.levels, prm.n_levels, prm.auto_reset, prm.seed, prm.env_offset + e, prm.counters, jab);
        K2D_PHASE(PH_EPILOGUE);
    }

    // ---- whole launch for one scene
    // steps s0 .. s1-1 of env e.  The state record may have been written by another SM earlier in this
    // launch, so it is read past the (non-coherent) L1.
    // e_in < 0: this group has no env in the current batch.  n_sync: the steps every group of the batch goes through; after
    // each of them the warps that share a scheduler meet at the named barrier `bar` (BAR_THREADS threads; none when a warp is
    // alone on its barrier), so that they run the same phase of a step at about the same time and share its instructions.
    template <int BAR_THREADS>
    __device__ __forceinline__ void run(int e_in, int s0, int s1, int n_sync, int bar) {
        const bool has = e_in >= 0;
        const int e = has ? e_in : 0;
        uint32_t *st = prm.state + (size_t)e * SC::ST_WORDS;
        K2D_PHASE_BEGIN();
        if (has) {
        // everything the state record holds for this lane is asked for in one go (the warm list entries are read a little
        // past the count, inside the record, and dropped below), then the level's constants in a second go
        constexpr int KB = (6 * SC::N + G - 1) / G;
        uint32_t body[KB], meta = 0u, jacc[3] = { 0u, 0u, 0u }, wrm[kWarmWords];
#pragma unroll
        for (int k = 0; k < KB; ++k) { const int i = lane + k * G; body[k] = (i < 6 * SC::N) ? __ldcg(st + SC::ST_BODY + i) : 0u; }
        if (lane < 5) meta = __ldcg(st + SC::ST_META + lane);
        if (SC::J > 0 && lane < SC::J) {
#pragma unroll
            for (int q = 0; q < 3; ++q) jacc[q] = __ldcg(st + SC::ST_JACC + 3 * lane + q);
        }
#pragma unroll
        for (int q = 0; q < kWarmWords; ++q) wrm[q] = (lane < SC::NPAIRS) ? __ldcg(st + SC::ST_WARM + kWarmWords * lane + q) : 0u;
        const int level = ck_idx<CK_LEVEL_ID>((int)__ldcg(st + SC::ST_META + META_LEVEL), prm.n_levels);
        const int nwarm = ck_idx<CK_COUNT>((int)__ldcg(st + SC::ST_META + META_NWARM), SC::NPAIRS + 1);
#pragma unroll
        for (int k = 0; k < KB; ++k) { const int i = lane + k * G; if (i < 6 * SC::N) smu[body_word<SC>(i)] = body[k]; }
        if (lane < 5) smu[SC::META + lane] = meta;
        if (SC::J > 0 && lane < SC::J) {
            smu[SC::JROW + kJointWords * lane + JR_ACCX] = jacc[0];
            smu[SC::JROW + kJointWords * lane + JR_ACCY] = jacc[1];
            smu[SC::JROW + kJointWords * lane + JR_ACCR] = jacc[2];
        }
        for (int i = lane; i < (SC::NPAIRS + 3) / 4; i += G) smu[SC::WIDX + i] = 0xffffffffu;
        jab = load_level_consts<SC, G>(smu, prm.levels + (size_t)level * SC::LV_WORDS);
        g.sync();
        // accumulated impulses of the previous launch: entry k goes to lane k
        rec.ab = 0u; rec.accn = 0.0f; rec.acct = 0.0f;
        lanef(LF_ACC2N) = 0.0f; lanef(LF_ACC2T) = 0.0f;
        if (lane < nwarm) {
            const uint32_t p = wrm[0];
            rec.ab = p << 12;
            rec.accn = __uint_as_float(wrm[1]); rec.acct = __uint_as_float(wrm[2]);
            lanef(LF_ACC2N) = __uint_as_float(wrm[3]); lanef(LF_ACC2T) = __uint_as_float(wrm[4]);
            widx()[ck_idx<CK_PAIR>((int)p, SC::NPAIRS)] = (uint8_t)lane;
        }
        if (lane < G / 2 && G + lane < nwarm) {
            const uint32_t *wr = st + SC::ST_WARM + kWarmWords * (G + lane);
            const uint32_t p = __ldcg(wr);
            ovl(R_AB) = __uint_as_float(p << 12);
            ovl(OV_ACC0N) = __uint_as_float(__ldcg(wr + 1)); ovl(OV_ACC0T) = __uint_as_float(__ldcg(wr + 2));
            ovl(OV_ACC1N) = __uint_as_float(__ldcg(wr + 3)); ovl(OV_ACC1T) = __uint_as_float(__ldcg(wr + 4));
            widx()[ck_idx<CK_PAIR>((int)p, SC::NPAIRS)] = (uint8_t)(G + lane);
        }
        if (nwarm > G + G / 2) warm_in<SC, G>(sm, ovf, st + SC::ST_WARM, nwarm);
        }
        g.sync();
        K2D_PHASE(PH_LOAD);
#pragma unroll 1
        for (int k = 0; k < n_sync; ++k) {
            const int s = s0 + k;
            if (has && s < s1) {
                step(e, s);
                if ((k & 255) == 255) flush();
            }
            g.sync();
            if (BAR_THREADS > 32) {
                __syncwarp();
                asm volatile("barrier.sync %0, %1;" :: "r"(bar), "r"(BAR_THREADS) : "memory");
            }
        }
        if (!has) return;
        K2D_PHASE_RESTART();
        // write back
        for (int i = lane; i < 6 * SC::N; i += G) st[SC::ST_BODY + i] = smu[body_word<SC>(i)];
        if (SC::J > 0 && lane < SC::J) {
            st[SC::ST_JACC + 3 * lane] = smu[SC::JROW + kJointWords * lane + JR_ACCX];
            st[SC::ST_JACC + 3 * lane + 1] = smu[SC::JROW + kJointWords * lane + JR_ACCY];
            st[SC::ST_JACC + 3 * lane + 2] = smu[SC::JROW + kJointWords * lane + JR_ACCR];
        }
        if (lane < 5) st[SC::ST_META + lane] = smu[SC::META + lane];
        const int nw = ck_idx<CK_COUNT>((int)smu[SC::META + META_NWARM], SC::NPAIRS + 1);
        if (lane < nw) {
            uint32_t *wr = st + SC::ST_WARM + kWarmWords * lane;
            wr[0] = (rec.ab >> 12) & 127u;
            wr[1] = __float_as_uint(rec.accn); wr[2] = __float_as_uint(rec.acct);
            wr[3] = __float_as_uint(lanef(LF_ACC2N)); wr[4] = __float_as_uint(lanef(LF_ACC2T));
        }
        if (lane < G / 2 && G + lane < nw) {
            uint32_t *wr = st + SC::ST_WARM + kWarmWords * (G + lane);
            wr[0] = (__float_as_uint(ovl(R_AB)) >> 12) & 127u;
            wr[1] = __float_as_uint(ovl(OV_ACC0N)); wr[2] = __float_as_uint(ovl(OV_ACC0T));
            wr[3] = __float_as_uint(ovl(OV_ACC1N)); wr[4] = __float_as_uint(ovl(OV_ACC1T));
        }
        if (nw > G + G / 2) warm_out<SC, G>(ovf, st + SC::ST_WARM, nw);
        g.sync();
        K2D_PHASE(PH_STORE);
        if (prm.obs && s1 == prm.n_steps) {
            ObsDims od; od.n_polygons = prm.n_polygons; od.n_circles = prm.n_circles; od.n_joints = prm.n_joints; od.n_thrusters = prm.n_thrusters; od.n_actions = prm.n_actions;
            write_obs<SC, G>(sm, prm.levels, prm.obs, od, e);
        }
    }
};

// ---------------------------------------------------------------- the order in which a launch hands out the envs
// The two scenes of a warp run in lockstep, so each pays for the longer of the two in every phase.  Handing out the envs
// sorted by what their steps cost puts like next to like: the key is the number of joint levels of the env's level and the
// number of pairs that were touching after its last step.  A counting sort in two launches: the first counts the keys and
// its last block turns the counts into first positions; the second writes every env to a position of its key.  The order
// inside a key is whatever the atomics give; no result depends on it.  sort[0 .. 255] counts (zero between launches),
// sort[256 .. 511] positions, sort[512] blocks that have counted.
constexpr int kOrderThreads = 256, kOrderKeys = 256;
template <class SC>
__device__ __forceinline__ int order_key(const uint32_t *state, const uint32_t *levels, int e, int n_levels) {
    const uint32_t *st = state + (size_t)e * SC::ST_WORDS;
    const unsigned level = min(__ldcg(st + SC::ST_META + META_LEVEL), (unsigned)(n_levels - 1));
    const unsigned touching = min(__ldcg(st + SC::ST_META + META_NWARM), 31u);
    const unsigned joint_levels = (__ldg(levels + (size_t)level * SC::LV_WORDS + SC::LV_GB) >> 24) & 7u;
    return kOrderKeys - 1 - (int)(joint_levels * 32u + touching);     // costly envs first: the cheap ones fill the end of the launch
}
template <class SC>
__global__ void __launch_bounds__(kOrderThreads) k2d_order_count_kernel(const uint32_t *state, const uint32_t *levels, unsigned int *sort,
                                                                        int n_envs, int n_levels) {
    __shared__ unsigned int s_cnt[kOrderKeys];
    __shared__ bool s_last;
    s_cnt[threadIdx.x] = 0u;
    __syncthreads();
    const int e = blockIdx.x * kOrderThreads + threadIdx.x;
    if (e < n_envs) atomicAdd(&s_cnt[order_key<SC>(state, levels, e, n_levels)], 1u);
    __syncthreads();
    if (s_cnt[threadIdx.x]) atomicAdd(sort + threadIdx.x, s_cnt[threadIdx.x]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(sort + 2 * kOrderKeys, 1u) == gridDim.x - 1u;
    __syncthreads();
    if (!s_last) return;
    // the last block to arrive: counts -> first positions (exclusive sums), counts back to zero for the next launch
    __threadfence();
    const unsigned int mine = __ldcg(sort + threadIdx.x);
    s_cnt[threadIdx.x] = mine;
    __syncthreads();
    for (int d = 1; d < kOrderKeys; d <<= 1) {
        const unsigned int v = threadIdx.x >= d ? s_cnt[threadIdx.x - d] : 0u;
        __syncthreads();
        s_cnt[threadIdx.x] += v;
        __syncthreads();
    }
    sort[kOrderKeys + threadIdx.x] = s_cnt[threadIdx.x] - mine;
    sort[threadIdx.x] = 0u;
    if (threadIdx.x == 0) sort[2 * kOrderKeys] = 0u;
}
template <class SC>
__global__ void __launch_bounds__(kOrderThreads) k2d_order_place_kernel(const uint32_t *state, const uint32_t *levels, unsigned int *sort,
                                                                        int *order, int n_envs, int n_levels) {
    const int e = blockIdx.x * kOrderThreads + threadIdx.x;
    if (e >= n_envs) return;
    const unsigned int pos = atomicAdd(sort + kOrderKeys + order_key<SC>(state, levels, e, n_levels), 1u);
    if (pos < (unsigned)n_envs) order[pos] = e;
}

template <class SC>
__device__ __forceinline__ uint16_t pair_code(int p) {
    int a, b;
    if (p < SC::NPP) { int i = 0, rem = p; while (rem >= SC::P - 1 - i) { rem -= SC::P - 1 - i; ++i; } a = i; b = i + 1 + rem; }
    else if (p < SC::NPP + SC::NPC) { const int q = p - SC::NPP; a = q / SC::C; b = SC::P + q % SC::C; }
    else { int i = 0, rem = p - SC::NPP - SC::NPC; while (rem >= SC::C - 1 - i) { rem -= SC::C - 1 - i; ++i; } a = SC::P + i; b = SC::P + i + 1 + rem; }
    return (uint16_t)(a | (b << 8));
}

// THREADS: kSmallBlock (several blocks per SM) or step_block_threads<SC, G>() (one block per SM).
template <class SC, int G, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == kSmallBlock ? kSmallBlocksPerSM : 1) k2d_step_kernel(const StepParams prm) {
    extern __shared__ __align__(16) uint32_t smem_raw[];
    constexpr int GPB = THREADS / G;
    uint16_t *ptab = reinterpret_cast<uint16_t *>(smem_raw);
    for (int p = threadIdx.x; p < SC::NPAIRS; p += THREADS) ptab[p] = pair_code<SC>(p);
    __syncthreads();
    const int gib = threadIdx.x / G;
    const int slot = blockIdx.x * GPB + gib, nslots = gridDim.x * GPB;
    uint32_t *region = smem_raw + SC::PTAB_WORDS + gib * region_words<SC, G>();
    uint32_t *scratch = prm.scratch + (size_t)ck_idx<CK_SLOT>(slot, prm.n_slots) * SC::SCRATCH_WORDS;
    Scene<SC, G> scene(region, ptab, scratch, prm);
    const Group<G> &g = scene.g;
    // Work items are (chunk, env), numbered in that order and dealt out in batches of kBatch consecutive ones to the warps of
    // the block that share a scheduler (warp number mod 4: WPS warps, kBatch scene groups), which step their scenes in
    // lockstep, a named barrier after every step: the warps of a scheduler then run the same phase of a step at about the
    // same time and fetch its instructions once.  With the envs sorted by cost the scenes of a batch are alike, so the
    // barriers wait little.  First batches go round the SMs (no ticket, and every SM starts with a mix of cheap and costly
    // envs); after that a leader draws the next batch number for its scheduler group from one ticket counter, so groups with
    // cheap scenes take more batches.  Chunk c of an env may start only when its chunk c - 1 is stepped and its state is
    // back in memory (another scheduler group may have done it); with batches handed out in order that is almost always
    // long past, else the group waits, with a limit, for the group that holds it, which is running.  Every thread of a
    // scheduler group goes through the same number of barriers: the batch number is the same for all of them, a batch takes
    // chunk_steps steps whether a group has an env in it or not, and a wait that runs out only turns the group's env off.
    constexpr int GPW = 32 / G, WPS = THREADS / 128, kBatch = WPS * GPW, BAR_THREADS = 32 * WPS;
    __shared__ unsigned int s_batch[4];
    const int warp = threadIdx.x >> 5, sub = warp & 3, bar = 1 + sub;
    const int member = (warp >> 2) * GPW + gib % GPW;
    const unsigned items = (unsigned)prm.n_envs * (unsigned)prm.n_chunks;
    const unsigned n_item_batches = (items + kBatch - 1) / kBatch, n_sched = gridDim.x * 4u;
    unsigned batch = (unsigned)sub * gridDim.x + blockIdx.x;
#pragma unroll 1
    for (;;) {
        if (batch >= n_item_batches) break;
        const unsigned t = batch * kBatch + member;
        int e = -1, c = 0;
        if (t < items) {
            c = (int)(t / (unsigned)prm.n_envs);
            const int idx = (int)(t - (unsigned)c * (unsigned)prm.n_envs);
            e = prm.order ? ck_idx<CK_COUNT>(__ldg(prm.order + idx), prm.n_envs) : idx;
        }
        bool ok = true;
        if (e >= 0 && c > 0) {
            if (g.lane == 0) {
                const volatile unsigned int *flag = prm.chunks_done + e;
                const volatile unsigned int *err = prm.queue + Q_ERROR;
                unsigned polls = 0u;
                while (*flag != (unsigned)c) {
                    if (*err != 0u || ++polls > prm.wait_limit) { atomicExch(prm.queue + Q_ERROR, 1u); ok = false; break; }
                    __nanosleep(100);
                }
            }
            ok = g.shfl(ok ? 1 : 0, 0) != 0;
            __threadfence();
        }
        const int s0 = c * prm.chunk_steps;
        scene.template run<BAR_THREADS>(ok ? e : -1, s0, min(prm.n_steps, s0 + prm.chunk_steps), prm.chunk_steps, bar);
        // the group's work counters go to the global ones every 64 steps or more (16-bit fields; a step adds at most
        // one manifold per slot, 186, and a run flushes every 256 steps by itself: (63 + 256) x 186 < 65536)
        if ((scene.c_man >> 16) >= 64u) scene.flush();
        if (e >= 0 && prm.n_chunks > 1) {
            __threadfence();      // this lane's part of the state record is visible before the count moves
            g.sync();
            if (g.lane == 0) atomicExch(prm.chunks_done + e, (c + 1 == prm.n_chunks) ? 0u : (unsigned)(c + 1));
        }
        // the next batch of this scheduler group
        if (warp < 4 && (threadIdx.x & 31) == 0) s_batch[sub] = n_sched + atomicAdd(prm.queue + Q_TICKET, 1u);
        if (BAR_THREADS > 32) { __syncwarp(); asm volatile("barrier.sync %0, %1;" :: "r"(bar), "r"(BAR_THREADS) : "memory"); }
        else __syncwarp();
        batch = s_batch[sub];
        if (BAR_THREADS > 32) { __syncwarp(); asm volatile("barrier.sync %0, %1;" :: "r"(bar), "r"(BAR_THREADS) : "memory"); }
        else __syncwarp();
    }
    scene.flush();
    // the last group to leave rewinds the queue for the next launch
    if (g.lane == 0) {
        __threadfence();
        if (atomicAdd(prm.queue + Q_LEFT, 1u) == (unsigned)nslots - 1u) {
            atomicExch(prm.queue + Q_TICKET, 0u);
            atomicExch(prm.queue + Q_LEFT, 0u);
        }
    }
}

// ---------------------------------------------------------------- reset kernel: one thread per (env, word)
template <class SC>
__global__ void k2d_reset_kernel(uint32_t *state, const uint32_t *levels, const int *level_ids, int n_envs, int n_levels) {
    const int e = blockIdx.x;
    if (e >= n_envs) return;
    const int l = level_ids ? level_ids[e] : e % n_levels;
    uint32_t *st = state + (size_t)e * SC::ST_WORDS;
    const uint32_t *lv = levels + (size_t)l * SC::LV_WORDS;
    for (int i = threadIdx.x; i < SC::ST_WARM; i += blockDim.x) {
        uint32_t v = 0u;
        if (i < 6 * SC::N) v = lv[SC::LV_X + i];
        else if (i == SC::ST_META + 2) v = (uint32_t)l;
        st[i] = v;
    }
}

// ---------------------------------------------------------------- observation kernel: one half-warp per env
// The 16 lanes of an env first ask for every word of the state record and of the level record that their rows need (lane l:
// shape l, joint side l, thruster l - 12), clear the env's shared-memory image of the observation while the loads are in
// flight, then write one shape row each, then one joint side or thruster row each, and copy the image out with coalesced
// stores.  Two envs share every instruction of a warp.
static_assert(K2D_MAX_SHAPES <= 16 && 2 * K2D_MAX_JOINTS <= 12 && K2D_MAX_THRUSTERS <= 4, "observation rows: one lane of sixteen each");
constexpr int kObsEnvsPerBlock = 2 * (kObsThreads / 32);
// words between the images of two envs: room for the rows and the cos / sin table, a multiple of 4, and 16 past a multiple of
// 32 so that the row stores of a warp's two envs (rows 29 or an odd number of words apart) fall into different banks
__host__ __device__ inline int obs_image_stride(int width, int n_bodies) {
    const int s = (width + 2 * n_bodies + 3) / 4 * 4;
    return s + (48 - s % 32) % 32;
}
template <class SC>
__global__ void __launch_bounds__(kObsThreads) k2d_obs_kernel(const uint32_t *state, const uint32_t *levels, float *obs,
                                                              int n_envs, int n_actions, int n_polygons, int n_circles,
                                                              int n_joints, int n_thrusters) {
    extern __shared__ __align__(16) float obs_smem[];
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31, half = lane >> 4, hl = lane & 15;
    const int e = blockIdx.x * kObsEnvsPerBlock + 2 * w + half;
    if (blockIdx.x * kObsEnvsPerBlock + 2 * w >= n_envs) return;     // the whole warp is past the last env
    const bool live = e < n_envs;
    const int n_shapes = n_polygons + n_circles;
    const int jw = 11 + n_actions;
    const int width = n_shapes * 29 + 2 * n_joints * jw + 6 * n_thrusters;
    float *img = obs_smem + (size_t)(2 * w + half) * obs_image_stride(width, SC::N);
    float *cs = img + width;                 // cos, sin of every shape's angle
    const uint32_t *st = state + (size_t)(live ? e : 0) * SC::ST_WORDS;
    const float *stf = reinterpret_cast<const float *>(st);
    // the state words of this lane's shape do not wait for the level id
    const bool shape_lane = live && hl < n_shapes;
    const int i = shape_lane ? (hl < n_polygons ? hl : SC::P + (hl - n_polygons)) : 0;     // internal shape index
    float sx = 0.0f, sy = 0.0f, sth = 0.0f, svx = 0.0f, svy = 0.0f, sw = 0.0f;
    if (shape_lane) { sx = stf[i]; sy = stf[SC::N + i]; sth = stf[2 * SC::N + i]; svx = stf[3 * SC::N + i]; svy = stf[4 * SC::N + i]; sw = stf[5 * SC::N + i]; }
    const uint32_t *lv = levels + (size_t)st[SC::ST_META + META_LEVEL] * SC::LV_WORDS;
    const float *lvf = reinterpret_cast<const float *>(lv);
    const bool poly = i < SC::P;
    uint32_t fl = 0u;
    float c_im = 0.0f, c_ii = 0.0f, c_de = 0.0f, c_fr = 0.0f, c_re = 0.0f, c_rad = 0.0f, pv[8] = { 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f };
    const int j = hl >> 1, d = hl & 1;                                     // joint side
    const bool joint_lane = live && hl < 2 * n_joints;
    const int t = hl - 12;                                                 // thruster
    const bool thr_lane = live && t >= 0 && t < n_thrusters;
    uint32_t rw[8] = { 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u };                 // joint: packed word, anchors, speed, power, kind; thruster: its record
    if (shape_lane) {
        fl = __ldg(lv + SC::LV_FLAGS + i);
        c_im = __ldg(lvf + SC::LV_IM + i); c_ii = __ldg(lvf + SC::LV_II + i); c_de = __ldg(lvf + SC::LV_DENS + i);
        c_fr = __ldg(lvf + SC::LV_FR + i); c_re = __ldg(lvf + SC::LV_RE + i);
        if (poly) {
#pragma unroll
            for (int k = 0; k < 4; ++k) { pv[2 * k] = __ldg(lvf + SC::LV_PVX + 4 * i + k); pv[2 * k + 1] = __ldg(lvf + SC::LV_PVY + 4 * i + k); }
        } else c_rad = __ldg(lvf + SC::LV_RAD + (i - SC::P));
    }
    if (joint_lane) {
        const uint32_t *src = lv + SC::LV_JOINT + kJointLevelWords * j;
#pragma unroll
        for (int q = 0; q < 7; ++q) rw[q] = __ldg(src + q);
        rw[7] = __ldg(src + 10);
    } else if (thr_lane) {
        const uint32_t *src = lv + SC::LV_THR + 8 * t;
#pragma unroll
        for (int q = 0; q < 6; ++q) rw[q] = __ldg(src + q);
    }
    // absent entities and unset columns are zero
    if (live) {
        float4 *z = reinterpret_cast<float4 *>(img);
        for (int q = hl; q < (width + 3) / 4; q += 16) z[q] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    }
    __syncwarp();
    if (shape_lane) {
        float c, sn;
        sincos_spec(sth, c, sn);
        cs[i] = c; cs[SC::N + i] = sn;
        if (fl & F_ACTIVE) {
            float *o = img + hl * 29;
            const int nv = flag_nverts(fl);
            const uint32_t role = flag_role(fl);
            o[0] = sx; o[1] = sy; o[2] = svx; o[3] = svy;
            o[4] = c_im; o[5] = c_ii; o[6] = c_de;
            o[7] = tanh_spec(sw * 0.1f);
            o[8 + role] = 1.0f;
            o[12] = sn; o[13] = c; o[14] = c_fr; o[15] = c_re;
            if (poly) {
                o[16] = 1.0f;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (k < nv) { o[19 + 2 * k] = pv[2 * k]; o[20 + 2 * k] = pv[2 * k + 1]; }
                }
                o[nv == 3 ? 27 : 28] = 1.0f;
            } else {
                o[17] = 1.0f; o[18] = c_rad;
            }
        }
    }
    __syncwarp();
    if (joint_lane) {
        const uint32_t jab = rw[0];
        if ((jab >> 28) & 1u) {
            float *o = img + n_shapes * 29 + hl * jw;
            const int a = jab & 255, b = (jab >> 8) & 255;
            const int from = d ? b : a, to = d ? a : b;
            o[0] = 1.0f; o[1] = (rw[7] & 1u) ? 1.0f : 0.0f;
            // anchor on the "from" shape, then on the "to" shape
            o[2] = __uint_as_float(d ? rw[3] : rw[1]); o[3] = __uint_as_float(d ? rw[4] : rw[2]);
            o[4] = __uint_as_float(d ? rw[1] : rw[3]); o[5] = __uint_as_float(d ? rw[2] : rw[4]);
            o[6] = __uint_as_float(rw[6]); o[7] = __uint_as_float(rw[5]);
            const int bind = (int)((jab >> 16) & 255);
            if (bind < n_actions) o[9 + bind] = 1.0f;
            o[9 + n_actions] = __fmaf_rn(cs[SC::N + to], cs[from], -(cs[to] * cs[SC::N + from]));
            o[10 + n_actions] = __fmaf_rn(cs[to], cs[from], cs[SC::N + to] * cs[SC::N + from]);
        }
    } else if (thr_lane) {
        const uint32_t tp = rw[0];
        if ((tp >> 20) & 1u) {
            float *o = img + n_shapes * 29 + 2 * n_joints * jw + t * 6;
            const int k = tp & 255;
            float dx, dy;
            rot2(cs[k], cs[SC::N + k], __uint_as_float(rw[3]), __uint_as_float(rw[4]), dx, dy);
            o[0] = 1.0f; o[1] = __uint_as_float(rw[1]); o[2] = __uint_as_float(rw[2]); o[3] = __uint_as_float(rw[5]);
            o[4] = dy; o[5] = dx;
        }
    }
    __syncwarp();
    if (!live) return;
    float *out = obs + (size_t)e * width;
    if (((width & 3) == 0) && ((reinterpret_cast<uintptr_t>(obs) & 15) == 0)) {
        const float4 *src = reinterpret_cast<const float4 *>(img);
        float4 *dst = reinterpret_cast<float4 *>(out);
        for (int q = hl; q < width / 4; q += 16) dst[q] = src[q];
    } else {
        for (int q = hl; q < width; q += 16) out[q] = img[q];
    }
}

// ---------------------------------------------------------------- pixel observation: one block per env
// A 125 x 125 RGBA image of the scene: the centre of pixel (row r, column c) is the world point
// (-3.125 + (c + 0.5) * 0.05, 5.75 - (r + 0.5) * 0.05); a pixel takes the colour of the highest-index active
// shape that contains its centre (polygon: not outside any face; circle: squared distance <= radius squared),
// white otherwise.
constexpr int kPix = 125;
constexpr int kRenderThreads = 128;
// pixel columns and rows that certainly cover a world-frame box (one pixel and 1 cm to spare); the exact tests decide
__device__ __forceinline__ int4 pixel_range(float x0, float y0, float x1, float y1) {
    const int c_lo = (int)fmax_cmp(fmin_cmp((x0 - 0.01f + 3.125f) * 20.0f - 1.5f, 126.0f), 0.0f);
    const int c_hi = (int)fmax_cmp(fmin_cmp((x1 + 0.01f + 3.125f) * 20.0f + 1.5f, 124.0f), -1.0f);
    const int r_lo = (int)fmax_cmp(fmin_cmp((5.75f - (y1 + 0.01f)) * 20.0f - 1.5f, 126.0f), 0.0f);
    const int r_hi = (int)fmax_cmp(fmin_cmp((5.75f - (y0 - 0.01f)) * 20.0f + 1.5f, 124.0f), -1.0f);
    return make_int4(c_lo, c_hi, r_lo, r_hi);
}
template <class SC>
__global__ void __launch_bounds__(kRenderThreads) k2d_render_kernel(const uint32_t *state, const uint32_t *levels, uint32_t *pixels, int n_envs) {
    __shared__ int4 s_rng[SC::N];            // first and last column, first and last row that the shape's box can reach (culling only)
    __shared__ float4 s_nx[SC::N], s_ny[SC::N], s_off[SC::N];   // polygon: face normals and offsets; circle: centre x, y, radius^2 in .x
    __shared__ uint32_t s_col[SC::N];
    __shared__ int s_nv[SC::N];              // vertices of a polygon, 0 for a circle, -1 for a shape that is not drawn
    __shared__ uint2 s_span[kRenderThreads * SC::N];         // per row of the block: (first column | columns - 1 << 8, colour) of every shape the row cuts
    __shared__ int s_nspan[kRenderThreads];
    const int e = blockIdx.x;
    if (e >= n_envs) return;
    const uint32_t *st = state + (size_t)e * SC::ST_WORDS;
    const uint32_t *lv = levels + (size_t)st[SC::ST_META + META_LEVEL] * SC::LV_WORDS;
    const float *stf = reinterpret_cast<const float *>(st);
    const float *lvf = reinterpret_cast<const float *>(lv);
    for (int i = threadIdx.x; i < SC::N; i += kRenderThreads) {
        const uint32_t fl = lv[SC::LV_FLAGS + i];
        int nv = -1;
        if (fl & F_ACTIVE) {
            const float x = stf[i], y = stf[SC::N + i];
            const uint32_t role = flag_role(fl);
            uint32_t rgb = role == 1u ? (200u << 8) : role == 2u ? (220u << 16) : role == 3u ? 220u : ((fl & F_DYNAMIC) ? 0x808080u : 0x404040u);
            s_col[i] = rgb | 0xff000000u;
            if (i < SC::P) {
                nv = (int)flag_nverts(fl);
                float c, sn;
                sincos_spec(stf[2 * SC::N + i], c, sn);
                float nxs[4] = { 0.0f, 0.0f, 0.0f, 0.0f }, nys[4] = { 0.0f, 0.0f, 0.0f, 0.0f }, offs[4] = { 0.0f, 0.0f, 0.0f, 0.0f };
                float x0 = 0.0f, y0 = 0.0f, x1 = 0.0f, y1 = 0.0f;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (k < nv) {
                        float rx, ry;
                        rot2(c, sn, lvf[SC::LV_PVX + 4 * i + k], lvf[SC::LV_PVY + 4 * i + k], rx, ry);
                        rot2(c, sn, lvf[SC::LV_PNX + 4 * i + k], lvf[SC::LV_PNY + 4 * i + k], nxs[k], nys[k]);
                        const float wx = rx + x, wy = ry + y;
                        offs[k] = dot2(nxs[k], nys[k], wx, wy);
                        if (k == 0) { x0 = x1 = wx; y0 = y1 = wy; }
                        else { x0 = fmin_cmp(x0, wx); x1 = fmax_cmp(x1, wx); y0 = fmin_cmp(y0, wy); y1 = fmax_cmp(y1, wy); }
                    }
                }
                s_nx[i] = make_float4(nxs[0], nxs[1], nxs[2], nxs[3]); s_ny[i] = make_float4(nys[0], nys[1], nys[2], nys[3]);
                s_off[i] = make_float4(offs[0], offs[1], offs[2], offs[3]);
                s_rng[i] = pixel_range(x0, y0, x1, y1);
            } else {
                nv = 0;
                const float r = lvf[SC::LV_RAD + (i - SC::P)];
                s_nx[i] = make_float4(x, 0.0f, 0.0f, 0.0f); s_ny[i] = make_float4(y, 0.0f, 0.0f, 0.0f); s_off[i] = make_float4(r * r, 0.0f, 0.0f, 0.0f);
                s_rng[i] = pixel_range(x - r, y - r, x + r, y + r);
            }
        }
        s_nv[i] = nv;
    }
    __syncthreads();
    // A warp paints 32 consecutive rows in three passes.  First the (shape, row) pairs whose row the shape's box reaches are
    // numbered (shape-major) and dealt out to the lanes, 32 at a time: from the shape's faces (or its circle) a lane works out
    // between which columns the row can cut the shape, and pins down the first and the last column that are inside with the
    // exact inside test (the one that defines the image) on the few columns at either end of that span, where rounding could
    // matter; the columns in between are inside (the shapes are convex).  The result goes to the slot of (row, shape).  Then
    // every lane takes one row and packs its slots into a short list of (first column, last column, colour) in shape order.
    // Then the warp writes the rows one after the other, lane l the columns l, l + 32, l + 64, l + 96: a pixel takes the
    // colour of the last entry of its row's list that covers it, white if none does.
    static_assert(SC::N <= 16, "one lane of sixteen per shape");
    constexpr uint32_t kNoSpan = 0xffffffffu;
    __shared__ int s_first[kRenderThreads / 32][SC::N + 1];      // per warp: number of the first pair of every shape, and the total
    __shared__ int s_row0[kRenderThreads / 32][SC::N];          // per warp: first of the warp's rows that the shape's box reaches
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int R0 = 32 * warp, R1 = min(R0 + 31, kPix - 1);
    {
        int cnt = 0, row0 = 0;
        if (lane < SC::N && s_nv[lane] >= 0) {
            const int4 rng = s_rng[lane];
            row0 = max(rng.z, R0);
            cnt = max(min(rng.w, R1) - row0 + 1, 0);
        }
        int incl = cnt;
#pragma unroll
        for (int d = 1; d < 16; d <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl, d); if (lane >= d) incl += v; }
        if (lane < SC::N) { s_first[warp][lane] = incl - cnt; s_row0[warp][lane] = row0; }
        if (lane == SC::N - 1) s_first[warp][SC::N] = incl;
    }
    __syncwarp();
    const int n_pairs = s_first[warp][SC::N];
#pragma unroll 1
    for (int base = 0; base < n_pairs; base += 32) {
        const int item = base + lane;
        if (item >= n_pairs) continue;
        // the shape of the pair: the last one whose first pair is not after this one (shapes without pairs share their successor's number)
        int i = 0;
#pragma unroll
        for (int step = 8; step >= 1; step >>= 1) if (i + step < SC::N && s_first[warp][i + step] <= item) i += step;
        const int r = s_row0[warp][i] + (item - s_first[warp][i]);
        uint2 *slot = s_span + (size_t)(r * SC::N + i);
        const int nv = s_nv[i];
        const int4 rng = s_rng[i];
        const float py = 5.75f - ((float)r + 0.5f) * 0.05f;
        const float4 nx = s_nx[i], ny = s_ny[i], off = s_off[i];
        float lo = -1.0e9f, hi = 1.0e9f;      // world x between which the row can be inside the shape
        bool all_exact = false, none = false;
        float t0 = 0.0f, t1 = 0.0f, t2 = 0.0f, t3 = 0.0f, dy2 = 0.0f;
        if (nv > 0) {
            t0 = ny.x * py; t1 = ny.y * py; t2 = ny.z * py; t3 = ny.w * py;
            const float a[4] = { nx.x, nx.y, nx.z, nx.w }, c[4] = { t0 - off.x, t1 - off.y, t2 - off.z, t3 - off.w };
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (k < nv) {
                    if (fabsf(a[k]) < 1.0e-3f) {          // a face nearly along the row: it is out, not binding, or too close to call
                        if (c[k] > 1.0e-3f) none = true;
                        else if (c[k] > -1.0e-3f) all_exact = true;
                    } else {
                        const float bound = __fdividef(-c[k], a[k]);      // an estimate is enough: the exact test decides the ends of the span
                        if (a[k] > 0.0f) hi = fmin_cmp(hi, bound); else lo = fmax_cmp(lo, bound);
                    }
                }
            }
        } else {
            const float dy = py - ny.x;
            dy2 = dy * dy;
            const float h2 = off.x - dy2;
            if (h2 < -1.0e-4f) none = true;
            else { const float h = sqrtf(fmax_cmp(h2, 0.0f)); lo = nx.x - h; hi = nx.x + h; }
        }
        if (none || hi < lo - 0.2f) { slot->x = kNoSpan; continue; }
        // columns: pixel c has its centre at x = -3.125 + (c + 0.5) * 0.05
        const float clo = fmax_cmp((lo + 3.125f) * 20.0f - 0.5f, -4.0f), chi = fmin_cmp((hi + 3.125f) * 20.0f - 0.5f, 130.0f);
        const int c_first = max(max((int)floorf(clo) - 2, rng.x), 0), c_last = min(min((int)ceilf(chi) + 2, rng.y), kPix - 1);
        // columns sure_first .. sure_last are inside without a test (none if a face is too close to call)
        const int sure_first = all_exact ? c_last + 1 : max((int)ceilf(clo) + 2, c_first), sure_last = all_exact ? c_first - 1 : min((int)floorf(chi) - 2, c_last);
        auto exact = [&](int c) -> bool {
            const float px = -3.125f + ((float)c + 0.5f) * 0.05f;
            if (nv > 0)
                return !(__fmaf_rn(nx.x, px, t0) - off.x > 0.0f) && !(__fmaf_rn(nx.y, px, t1) - off.y > 0.0f) &&
                       !(__fmaf_rn(nx.z, px, t2) - off.z > 0.0f) && (nv < 4 || !(__fmaf_rn(nx.w, px, t3) - off.w > 0.0f));
            const float dx = px - nx.x;
            return __fmaf_rn(dx, dx, dy2) <= off.x;
        };
        const bool sure = sure_first <= sure_last;
        int cf = sure ? sure_first : c_last + 1, cl = sure ? sure_last : c_first - 1;
        // the first inside column: the lowest one below the sure span (or anywhere, if there is no sure span) that passes the test
        const int left_end = sure ? sure_first - 1 : c_last;
#pragma unroll 1
        for (int c = c_first; c <= left_end; ++c) if (exact(c)) { cf = c; break; }
        const int right_end = sure ? sure_last + 1 : max(cf, c_first);
#pragma unroll 1
        for (int c = c_last; c >= right_end; --c) if (exact(c)) { cl = c; break; }
        if (!sure && cl < cf) cl = cf;      // a single column found from the left
        if (cf <= cl && cf <= c_last) *slot = make_uint2((uint32_t)cf | ((uint32_t)(cl - cf) << 8), s_col[i]);
        else slot->x = kNoSpan;
    }
    __syncwarp();
    // the slots of a row, packed in place (the list is never ahead of the slot being read)
    uint2 *spans = s_span + (warp * 32 + lane) * SC::N;
    const int r = R0 + lane;
    int n_span = 0;
    if (r < kPix) {
#pragma unroll 1
        for (int i = 0; i < SC::N; ++i) {
            if (s_nv[i] < 0) continue;
            const int4 rng = s_rng[i];
            if (r < rng.z || r > rng.w) continue;
            const uint2 w = spans[i];
            if (w.x != kNoSpan) spans[n_span++] = w;
        }
    }
    s_nspan[warp * 32 + lane] = n_span;
    __syncwarp();
    const int n_rows = min(32, kPix - 32 * warp);
    uint32_t *img = pixels + (size_t)e * kPix * kPix + (size_t)warp * 32 * kPix;
#pragma unroll 1
    for (int j = 0; j < n_rows; ++j) {
        const int ns = s_nspan[warp * 32 + j];
        const uint2 *sp = s_span + (warp * 32 + j) * SC::N;
        uint32_t col[4] = { 0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu };
#pragma unroll 1
        for (int k = 0; k < ns; ++k) {
            const uint2 w = sp[k];
            const unsigned cf = w.x & 255u, len = w.x >> 8;
            const unsigned d = (unsigned)lane - cf;          // column - first column, for the lane's four columns d, d + 32, ...
#pragma unroll
            for (int q = 0; q < 4; ++q) if (d + 32u * q <= len) col[q] = w.y;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) if (32 * q + lane < kPix) img[j * kPix + 32 * q + lane] = col[q];
    }
}

__global__ void k2d_eval_kernel(const float *x, int n, float *c, float *s, float *t) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float cc, ss;
    sincos_spec(x[i], cc, ss);
    if (c) c[i] = cc;
    if (s) s[i] = ss;
    if (t) t[i] = tanh_spec(x[i]);
}

// ---------------------------------------------------------------- FP32 throughput probe
// Eight independent chains of fused multiply-adds per thread, kFmaChainSteps links each: what the FP32 pipes of the device
// sustain when nothing else limits them.  The result is stored so that the chains are not removed.
constexpr int kFmaChainSteps = 4096, kFmaChains = 8;
__global__ void __launch_bounds__(256) k2d_fma_chain_kernel(float *out, float a, float b) {
    float v[kFmaChains];
#pragma unroll
    for (int k = 0; k < kFmaChains; ++k) v[k] = (float)(threadIdx.x + k) * 1e-3f;
#pragma unroll 1
    for (int i = 0; i < kFmaChainSteps; i += 4) {
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int k = 0; k < kFmaChains; ++k) v[k] = __fmaf_rn(v[k], a, b);
    }
    float sum = 0.0f;
#pragma unroll
    for (int k = 0; k < kFmaChains; ++k) sum += v[k];
    out[blockIdx.x * blockDim.x + threadIdx.x] = sum;
}

}  // namespace k2d
