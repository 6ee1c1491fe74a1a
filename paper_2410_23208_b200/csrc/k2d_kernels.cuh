// k2d_kernels.cuh -- device code of the batched 2D rigid-body environment step (sm_100a).
//
// One engine step of every env is two kernel launches.
//
//   k2d_prep_kernel   A group of G lanes (G = 16: two scenes per warp; 32: one warp per scene; 8: four per warp)
//                     takes one scene at a time from a ticket queue.  Its lanes work on bodies, polygon vertices,
//                     shape pairs (bounding-box test, narrowphase) and touching pairs (one per lane): gravity,
//                     world-frame geometry, motors, thrusters, joint pre-step, manifolds, touch flags, and the
//                     pre-step of every touching pair.  It leaves the step's constraint rows (one 112-byte row per
//                     touching pair, sorted by solver level, and one 96-byte row per joint) in the env's scratch
//                     area and the velocities in the env's state record.
//   k2d_solve_kernel  A group of 4 lanes (eight scenes per warp) runs the warm start, the solver iterations, the Euler
//                     step and the positional corrections over those rows, then the reward, the termination and the
//                     auto-reset.  Only the bodies' velocities (later positions) and the accumulated impulses are in
//                     shared memory; the rows' constants are read through the read-only cache.
//
// The sequential-impulse solver of a scene is a chain of dependent rows with two or three independent rows per link,
// so it can feed few lanes; its working set is small.  The geometry of a scene is wide (120 pairs to test for the
// largest size class) and needs a working set of several kilobytes in shared memory.  Hence two kernels with
// different lanes per scene and different occupancy.
//
// Arithmetic contract: every +,-,*,/,sqrt is an individually rounded IEEE binary32 operation
// (the file is compiled with --fmad=false --prec-div=true --prec-sqrt=true --ftz=false), a fused
// multiply-add appears only where the code says __fmaf_rn, and min/max are comparisons.  The solver visits
// rows in an order equivalent to the canonical one (joints by index, then touching pairs by pair index): "level
// scheduling": a row's level is one more than the highest level of an earlier row that shares a movable body with it;
// rows of one level touch disjoint movable bodies and run on different lanes at once, and levels run in order, so every
// body sees exactly the sequence of updates a one-row-at-a-time sweep would give it: results are bit-identical to that sweep.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace k2d {

#ifndef K2D_BLOCK_THREADS
#define K2D_BLOCK_THREADS 128
#endif
constexpr int kBlockThreads = K2D_BLOCK_THREADS;
#ifndef K2D_MIN_BLOCKS
#define K2D_MIN_BLOCKS 6
#endif
constexpr int kMinBlocks = K2D_MIN_BLOCKS;   // resident blocks per SM the prep kernel is compiled for (bounds its registers)
#ifndef K2D_SOLVE_THREADS
#define K2D_SOLVE_THREADS 64
#endif
constexpr int kSolveThreads = K2D_SOLVE_THREADS;
#ifndef K2D_SOLVE_LANES
#define K2D_SOLVE_LANES 4
#endif
constexpr int kSolveLanes = K2D_SOLVE_LANES;       // solve kernel: lanes per scene
constexpr int kObsThreads = 128;   // observation kernel: one warp per env, four envs per block
constexpr int kMaxActions = 16;
enum { Q_TICKET = 0, Q_LEFT = 1 };
constexpr int kRowWords = 28;   // one touching pair: seven 16-byte groups
constexpr int kWarmWords = 5;   // pair index + 4 accumulated impulses
constexpr int kStageWords = 9;  // packed pair word, normal, two contact points with penetration
constexpr int kStageStride = 12; // a staged pair in scratch: the stage words, then the row slot it is to fill
constexpr int kJointWords = 24; // joint row: six 16-byte groups
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
    // state record of an env: per body the 16-byte groups (x, y, angle, -) and (vx, vy, angular velocity, -), meta,
    // accumulated joint impulses, and the accumulated impulses of the manifolds that were active in the latest step
    static constexpr int ST_POS = 0, ST_VEL = 4 * N, ST_META = 8 * N, ST_JACC = ST_META + 8;
    static constexpr int ST_WARM = (ST_JACC + 3 * J + 3) / 4 * 4;
    static constexpr int ST_WORDS = (ST_WARM + kWarmWords * NPAIRS + 3) / 4 * 4;
    // scratch of an env, valid from the prep kernel of a step to its solve kernel: pair rows sorted by level, joint rows,
    // the first row of every level (bytes; entry L for level L, entry highest level + 1 = number of rows), and a
    // staging area for the pairs of a scene with more touching pairs than lanes
    static constexpr int SCR_ROWS = 0, SCR_JROW = NPAIRS * kRowWords;
    static constexpr int SCR_LSTART = SCR_JROW + kJointWords * J;
    static constexpr int SCR_STAGE = SCR_LSTART + ((NPAIRS + 2 + 3) / 4 + 3) / 4 * 4;
    static constexpr int SCRATCH_WORDS = SCR_STAGE + kStageStride * NPAIRS;
    // shared memory region of one scene in the prep kernel (words)
    // per body 16-byte groups (x, y, angle, -) and (vx, vy, angular velocity, -), then per-body arrays
    static constexpr int BPOS = 0, BVEL = 4 * N;
    static constexpr int BIM = 8 * N, BII = 9 * N, BFR = 10 * N, BRE = 11 * N, BC = 12 * N, BS = 13 * N, BFL = 14 * N;
    static constexpr int RAD = 15 * N;
    static constexpr int WVX = (RAD + C + 3) / 4 * 4, WVY = WVX + P4, WNX = WVY + P4, WNY = WNX + P4, WOFF = WNY + P4;
    static constexpr int BOX = (WOFF + P4 + 3) / 4 * 4;  // N x (min x, min y, max x, max y), 16-byte aligned
    static constexpr int MASK = BOX + 4 * N;
    static constexpr int ACT = MASK + MASKW;
    static constexpr int META = ACT + kMaxActions;       // the state record's meta words
    static constexpr int LVC = (META + 8 + 3) / 4 * 4;   // copy of the level record's edge lengths, joint and thruster records
    static constexpr int LVC_WORDS = LV_MASK - LV_ELEN;
    static constexpr int ELEN = LVC, LVC_JOINT = LVC + (LV_JOINT - LV_ELEN), LVC_THR = LVC + (LV_THR - LV_ELEN);
    static constexpr int SURV = LVC + LVC_WORDS;         // bytes: pairs that passed the box test; afterwards per-body words of the level search
    static constexpr int WIDX = SURV + ((NPAIRS + 3) / 4 > N ? (NPAIRS + 3) / 4 : N); // bytes: pair -> entry of the previous step's warm list
    // then, per lane of the group (field-major, G words per field): kStageWords fields, touching pairs on their way to
    // the lane that builds their rows
    static constexpr int STG = WIDX + (NPAIRS + 3) / 4;
    static constexpr int PTAB_WORDS = ((NPAIRS + 1) / 2 + 3) / 4 * 4;  // block-shared pair table, 16 bits per pair
};
// pair row (scratch): what the solver needs of one touching pair: pair word, normal, friction | inverse masses and inertias |
// per manifold the lever-arm cross products, effective masses, target normal velocity, positional correction | the four
// accumulated impulses
enum { R_AB = 0, R_NX, R_NY, R_MU, R_MA, R_MB, R_IA, R_IB, R_M0 = 8, R_M1 = 16, R_ACC = 24 };
enum { M_RNA = 0, M_RNB, M_RTA, M_RTB, M_MASSN, M_MASST, M_TARGET, M_CORR };
static_assert(R_ACC + 4 == kRowWords, "row size");
// row AB word = staged AB word
// staged manifold fields
enum { S_AB = 0, S_NX, S_NY, S_PX0, S_PY0, S_PEN0, S_PX1, S_PY1, S_PEN1 };
static_assert(S_PEN1 + 1 == kStageWords, "stage size");
// staged AB word: a | b<<5 | active manifolds<<10 | pair<<12 | level<<19 | a movable<<26 | b movable<<27
// joint row fields
enum { JR_RAX = 0, JR_RAY, JR_RBX, JR_RBY, JR_I11, JR_I12, JR_I22, JR_JAB, JR_BX, JR_BY, JR_CX, JR_CY, JR_MA, JR_MB, JR_IA, JR_IB,
       JR_ACCX, JR_ACCY, JR_PAD1, JR_PAD2,
       JR_ANG, JR_KR, JR_BIASR, JR_ACCR };   // angular row: kind (0 none, 1 fixed, 2 beyond the upper limit, 3 beyond the lower), 1 / (1/I_a + 1/I_b), gamma x error, accumulated
static_assert(JR_ACCR + 1 == kJointWords, "joint row size");
// meta words of a state record.  NROWS is the number of pair rows of the latest step (= entries of the warm list).  FLAGS, D0
// and ACTIVE are messages from the prep kernel to the solve kernel of the same step: touch flags (green-blue | green-red << 1),
// the dense reward's shapes (both exist << 2 | green << 8 | blue << 16), the highest contact level << 24; the distance of
// those shapes before the step; the bit mask of the shapes that exist | the highest joint level << 16.
enum { META_STEP = 0, META_EPISODE, META_LEVEL, META_STATUS, META_NROWS, META_FLAGS, META_D0, META_ACTIVE };

// shared-memory words per scene: padded so that the groups of one warp start in different banks
template <class SC, int G>
__host__ __device__ constexpr int region_words() {
    constexpr int raw = SC::STG + kStageWords * G;
    return G < 32 ? (raw - G + 31) / 32 * 32 + G : (raw + 3) / 4 * 4;
}

// body flag word
constexpr uint32_t F_ACTIVE = 1u, F_DYNAMIC = 2u;
__host__ __device__ inline uint32_t flag_role(uint32_t f) { return (f >> 2) & 3u; }
__host__ __device__ inline uint32_t flag_nverts(uint32_t f) { return (f >> 4) & 7u; }
// joint packed word: a | b<<8 | binding<<16 | on<<24 | level<<25 | active<<28 | a movable<<29 | b movable<<30 | fixed or limited<<31
// thruster packed word: shape | binding<<8 | on<<16 | level<<17 | active<<20

struct StepParams {
    uint32_t *state;
    const uint32_t *levels;
    const float *actions;      // the action row of this step, [n_envs][n_actions]
    float *reward;             // this step's [n_envs]
    uint8_t *done;
    unsigned long long *counters;
    unsigned int *queue;       // work queue words of the prep kernel: next ticket, groups that have left
    uint32_t *scratch;         // [n_envs][SCRATCH_WORDS]
    float *trace;
    int n_envs, n_actions, n_levels;
    int solver_iters, warm_start, auto_reset, max_episode_steps;
    int discrete;             // actions are int32 codes (multi-discrete action space) instead of floats
    float dense_kappa;        // coefficient of the dense reward (0 = off)
    float dt, gdt, contact_alpha, contact_beta, slop, rest_thr, face_tol, joint_alpha, joint_beta, joint_gamma, motor_rho, aabb_margin;
    unsigned long long seed;
    long long env_offset;
};

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
template <class SC>
__device__ __forceinline__ uint16_t pair_code(int p) {
    int a, b;
    if (p < SC::NPP) { int i = 0, rem = p; while (rem >= SC::P - 1 - i) { rem -= SC::P - 1 - i; ++i; } a = i; b = i + 1 + rem; }
    else if (p < SC::NPP + SC::NPC) { const int q = p - SC::NPP; a = q / SC::C; b = SC::P + q % SC::C; }
    else { int i = 0, rem = p - SC::NPP - SC::NPC; while (rem >= SC::C - 1 - i) { rem -= SC::C - 1 - i; ++i; } a = SC::P + i; b = SC::P + i + 1 + rem; }
    return (uint16_t)(a | (b << 8));
}

// ================================================================ rarely run code, kept out of line
// what the prep kernel reads of an env's meta words before it starts on the env
struct MetaHead { uint32_t level, status, nprev; };
__device__ __forceinline__ MetaHead load_meta_head(const uint32_t *st_meta) {
    const uint4 m = __ldcg(reinterpret_cast<const uint4 *>(st_meta));
    MetaHead h; h.level = m.z; h.status = m.w; h.nprev = __ldcg(st_meta + META_NROWS);
    return h;
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

// A scene with more touching pairs than lanes: one lane walks the staged pairs in the scratch (in staging order), gives
// each its level (into bits 19.. of its packed word) and its row slot (the word after the stage words), and fills the
// table of level starts.  Returns the highest level.  bl: N bytes of shared memory.
template <class SC>
__device__ __noinline__ int place_crowded_impl(uint32_t *scr, uint8_t *lstart, uint8_t *bl, int nrec) {
    uint32_t *stage = scr + SC::SCR_STAGE;
    int cmax = 0;
    for (int i = 0; i < SC::N; ++i) bl[i] = 0;
    for (int L = 0; L <= nrec + 1; ++L) lstart[L] = 0;
    for (int k = 0; k < nrec; ++k) {
        uint32_t *w = stage + (size_t)k * kStageStride;
        const uint32_t ab = w[S_AB];
        const int a = ab & 31, b = (ab >> 5) & 31;
        int lvl = 1;
        if ((ab >> 26) & 1u) lvl = max(lvl, bl[a] + 1);
        if ((ab >> 27) & 1u) lvl = max(lvl, bl[b] + 1);
        if ((ab >> 26) & 1u) bl[a] = (uint8_t)lvl;
        if ((ab >> 27) & 1u) bl[b] = (uint8_t)lvl;
        w[S_AB] = ab | ((uint32_t)lvl << 19);
        lstart[lvl] = (uint8_t)(lstart[lvl] + 1);
        cmax = max(cmax, lvl);
    }
    // counts -> starts; a cursor per level in the spare word of stage entry level - 1
    int run = 0;
    for (int L = 1; L <= cmax; ++L) {
        const int c = lstart[L];
        lstart[L] = (uint8_t)run;
        stage[(size_t)(L - 1) * kStageStride + kStageWords + 1] = (uint32_t)run;
        run += c;
    }
    lstart[cmax + 1] = (uint8_t)run;
    for (int k = 0; k < nrec; ++k) {
        uint32_t *w = stage + (size_t)k * kStageStride;
        const int lvl = (int)((w[S_AB] >> 19) & 127u);
        uint32_t *cur = stage + (size_t)(lvl - 1) * kStageStride + kStageWords + 1;
        w[kStageWords] = *cur;
        *cur = *cur + 1u;
    }
    return cmax;
}

// ---------------------------------------------------------------- first half of a step: one scene per group of G lanes
template <class SC, int G>
struct Scene {
    static_assert(SC::J <= G && SC::T <= G && kMaxActions <= 2 * G, "one lane per joint / thruster");
    static_assert(SC::NPAIRS < 255, "pair indices are bytes");
    float *sm;            // this scene's shared-memory region
    uint32_t *smu;
    const uint16_t *ptab; // block-shared pair table
    const StepParams &prm;
    Group<G> g;
    int lane;
    unsigned c_surv, c_rec, c_man;   // packed work counters: pp | pc << 16, cc | active pairs << 16, manifolds | env-steps << 16

    __device__ __forceinline__ Scene(uint32_t *region, const uint16_t *pt, const StepParams &p)
        : sm(reinterpret_cast<float *>(region)), smu(region), ptab(pt), prm(p), g() {
        lane = g.lane; c_surv = 0u; c_rec = 0u; c_man = 0u;
    }

    __device__ __forceinline__ uint8_t *surv() { return reinterpret_cast<uint8_t *>(smu + SC::SURV); }
    __device__ __forceinline__ uint8_t *widx() { return reinterpret_cast<uint8_t *>(smu + SC::WIDX); }
    __device__ __forceinline__ float4 &box4(int i) { return *reinterpret_cast<float4 *>(sm + SC::BOX + 4 * i); }
    __device__ __forceinline__ ContactConsts contact_consts() const {
        ContactConsts cc; cc.slop = prm.slop; cc.rest_thr = prm.rest_thr; cc.alpha = prm.contact_alpha; cc.beta = prm.contact_beta; return cc;
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
                s = fmax_cmp(fmin_cmp(s, sm[SC::ELEN + 4 * a + k]), 0.0f);
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

    // ---- the first half of one environment step of env e (not frozen), whose meta head has been read already.
    // tn_raw: lane 0's ticket for the group's next env, still in flight; on return next_e is that ticket for all lanes
    // and next_head the env's meta head (if there is such an env), fetched while this env's pairs are tested.
    __device__ __forceinline__ void prepare(int e, const MetaHead &head, unsigned tn_raw, unsigned &next_e, MetaHead &next_head) {
        uint32_t *st = prm.state + (size_t)e * SC::ST_WORDS;
        uint32_t *scr = prm.scratch + (size_t)e * SC::SCRATCH_WORDS;
        const uint32_t *lv = prm.levels + (size_t)head.level * SC::LV_WORDS;
        const int nprev = (int)head.nprev;
        // Everything this step reads from memory is asked for here, in two volleys of loads that are all in flight before the
        // first of them is used, so that the group waits for memory twice per step and not once per word: the state record
        // (the same 16-byte groups as in shared memory), the level's constants, the body-frame vertices and normals (parked
        // where their world-frame images will go), the action row, the previous step's warm list.
        constexpr int KB = (2 * SC::N + G - 1) / G, KN = (SC::N + G - 1) / G, KV = (SC::P4 + G - 1) / G, KL = (SC::LVC_WORDS + G - 1) / G;
        {
            float4 body[KB];
            uint32_t cim[KN], cii[KN], cfr[KN], cre[KN], cfl[KN], pvx[KV], pvy[KV], pnx[KV], pny[KV];
#pragma unroll
            for (int k = 0; k < KB; ++k) { const int i = lane + k * G; body[k] = (i < 2 * SC::N) ? __ldcg(reinterpret_cast<const float4 *>(st + SC::ST_POS) + i) : make_float4(0.0f, 0.0f, 0.0f, 0.0f); }
#pragma unroll
            for (int k = 0; k < KN; ++k) {
                const int i = lane + k * G; const bool in = i < SC::N;
                cim[k] = in ? __ldg(lv + SC::LV_IM + i) : 0u; cii[k] = in ? __ldg(lv + SC::LV_II + i) : 0u; cfr[k] = in ? __ldg(lv + SC::LV_FR + i) : 0u;
                cre[k] = in ? __ldg(lv + SC::LV_RE + i) : 0u; cfl[k] = in ? __ldg(lv + SC::LV_FLAGS + i) : 0u;
            }
#pragma unroll
            for (int k = 0; k < KV; ++k) {
                const int v = lane + k * G; const bool in = v < SC::P4;
                pvx[k] = in ? __ldg(lv + SC::LV_PVX + v) : 0u; pvy[k] = in ? __ldg(lv + SC::LV_PVY + v) : 0u;
                pnx[k] = in ? __ldg(lv + SC::LV_PNX + v) : 0u; pny[k] = in ? __ldg(lv + SC::LV_PNY + v) : 0u;
            }
#pragma unroll
            for (int k = 0; k < KB; ++k) { const int i = lane + k * G; if (i < 2 * SC::N) reinterpret_cast<float4 *>(sm + SC::BPOS)[i] = body[k]; }
#pragma unroll
            for (int k = 0; k < KN; ++k) {
                const int i = lane + k * G;
                if (i < SC::N) { smu[SC::BIM + i] = cim[k]; smu[SC::BII + i] = cii[k]; smu[SC::BFR + i] = cfr[k]; smu[SC::BRE + i] = cre[k]; smu[SC::BFL + i] = cfl[k]; }
            }
#pragma unroll
            for (int k = 0; k < KV; ++k) {
                const int v = lane + k * G;
                if (v < SC::P4) { smu[SC::WVX + v] = pvx[k]; smu[SC::WVY + v] = pvy[k]; smu[SC::WNX + v] = pnx[k]; smu[SC::WNY + v] = pny[k]; }
            }
        }
        uint32_t gb;
        uint32_t wpair = 255u;
        float4 wacc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        float jacc0 = 0.0f, jacc1 = 0.0f, jacc2 = 0.0f;
        {
            uint32_t lvc[KL], rad = 0u, msk = 0u, act0 = 0u, act1 = 0u;
#pragma unroll
            for (int k = 0; k < KL; ++k) { const int i = lane + k * G; lvc[k] = (i < SC::LVC_WORDS) ? __ldg(lv + SC::LV_ELEN + i) : 0u; }
            static_assert(SC::C <= G && SC::MASKW <= G, "one lane per circle / mask word");
            if (lane < SC::C) rad = __ldg(lv + SC::LV_RAD + lane);
            if (lane < SC::MASKW) msk = __ldg(lv + SC::LV_MASK + lane);
            const uint32_t *act_row = reinterpret_cast<const uint32_t *>(prm.actions) + (size_t)e * prm.n_actions;
            if (lane < prm.n_actions) act0 = __ldg(act_row + lane);
            if (G < kMaxActions && lane + G < prm.n_actions) act1 = __ldg(act_row + lane + G);
            gb = __ldg(lv + SC::LV_GB);
            // the previous step's accumulated impulses: entry k stays with lane k (entries beyond the lanes are read from the
            // state record when needed); the byte table maps a pair to its entry
            if (lane < nprev) {
                const uint32_t *wr = st + SC::ST_WARM + kWarmWords * lane;
                wpair = __ldcg(wr);
                wacc = make_float4(__uint_as_float(__ldcg(wr + 1)), __uint_as_float(__ldcg(wr + 2)), __uint_as_float(__ldcg(wr + 3)), __uint_as_float(__ldcg(wr + 4)));
            }
            if (SC::J > 0 && lane < SC::J) {
                jacc0 = __uint_as_float(__ldcg(st + SC::ST_JACC + 3 * lane)); jacc1 = __uint_as_float(__ldcg(st + SC::ST_JACC + 3 * lane + 1));
                jacc2 = __uint_as_float(__ldcg(st + SC::ST_JACC + 3 * lane + 2));
            }
#pragma unroll
            for (int k = 0; k < KL; ++k) { const int i = lane + k * G; if (i < SC::LVC_WORDS) smu[SC::LVC + i] = lvc[k]; }
            if (lane < SC::C) smu[SC::RAD + lane] = rad;
            if (lane < SC::MASKW) smu[SC::MASK + lane] = msk;
            if (lane < prm.n_actions) smu[SC::ACT + lane] = act0;
            if (G < kMaxActions && lane + G < prm.n_actions) smu[SC::ACT + lane + G] = act1;
        }
        for (int i = lane; i < (SC::NPAIRS + 3) / 4; i += G) smu[SC::WIDX + i] = 0xffffffffu;
        g.sync();
        if (wpair != 255u) widx()[wpair] = (uint8_t)lane;
        for (int k = G + lane; k < nprev; k += G) widx()[__ldcg(st + SC::ST_WARM + kWarmWords * k)] = (uint8_t)k;
        const uint32_t jab = (SC::J > 0 && lane < SC::J) ? smu[SC::LVC_JOINT + kJointLevelWords * lane] : 0u;
        // dense reward: the first green and the first blue shape, and their distance before the step
        float d0 = 0.0f;
        if (prm.dense_kappa != 0.0f && ((gb >> 16) & 1u)) {
            const float4 pg = ld4(sm + SC::BPOS + 4 * (gb & 255u)), pb = ld4(sm + SC::BPOS + 4 * ((gb >> 8) & 255u));
            const float dx = pb.x - pg.x, dy = pb.y - pg.y;
            d0 = sqrtf(dot2(dx, dy, dx, dy));
        }
        // gravity, rotation, circle boxes
        unsigned active_mask = 0u;
        for (int base = 0; base < SC::N; base += G) {
            const int i = base + lane;
            bool act_i = false;
            if (i < SC::N) {
                const uint32_t fl = smu[SC::BFL + i];
                act_i = (fl & F_ACTIVE) != 0u;
                if (act_i && (fl & F_DYNAMIC)) sm[SC::BVEL + 4 * i + 1] = sm[SC::BVEL + 4 * i + 1] + prm.gdt;
                float c, sn;
                sincos_spec(sm[SC::BPOS + 4 * i + 2], c, sn);
                sm[SC::BC + i] = c; sm[SC::BS + i] = sn;
                if (i >= SC::P) {
                    const float r = sm[SC::RAD + (i - SC::P)], x = sm[SC::BPOS + 4 * i], y = sm[SC::BPOS + 4 * i + 1];
                    box4(i) = make_float4(x - r, y - r, x + r, y + r);
                }
            }
            active_mask |= g.ballot(act_i) << base;
        }
        g.sync();
        // world-frame polygon vertices, normals, face offsets (each lane turns the body-frame values it parked)
        for (int v = lane; v < SC::P4; v += G) {
            const int i = v >> 2, k = v & 3;
            if (k < (int)flag_nverts(smu[SC::BFL + i])) {
                const float c = sm[SC::BC + i], sn = sm[SC::BS + i];
                float rx, ry, nx, ny;
                rot2(c, sn, sm[SC::WVX + v], sm[SC::WVY + v], rx, ry);
                rot2(c, sn, sm[SC::WNX + v], sm[SC::WNY + v], nx, ny);
                const float wx = rx + sm[SC::BPOS + 4 * i], wy = ry + sm[SC::BPOS + 4 * i + 1];
                sm[SC::WVX + v] = wx; sm[SC::WVY + v] = wy; sm[SC::WNX + v] = nx; sm[SC::WNY + v] = ny;
                sm[SC::WOFF + v] = dot2(nx, ny, wx, wy);
            }
        }
        // this lane's joint: "on" bit and level come with the level record
        const bool jon = ((jab >> 24) & 1u) != 0u;
        const int jlevel = jon ? (int)((jab >> 25) & 7u) : 0;
        const int jmax = (SC::J > 0) ? g.max_int(jlevel) : 0;
        const uint32_t *jl = smu + SC::LVC_JOINT + kJointLevelWords * (lane < SC::J ? lane : 0);
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
        // motors in joint order: joints of one level touch disjoint movable shapes, levels in order keep the joint order
        if (SC::J > 0) {
#pragma unroll 1
            for (int lvl = 1; lvl <= jmax; ++lvl) {
                if (jlevel == lvl) {
                    const int a = jab & 255, b = (jab >> 8) & 255;
                    const float av = sm[SC::ACT + ((jab >> 16) & 255)];
                    // paper, "Action Space": continuous in [-1, 1], or multi-discrete codes 0 off, 1 forwards, 2 backwards at full power
                    const float A = prm.discrete ? (__float_as_int(av) == 1 ? 1.0f : (__float_as_int(av) == 2 ? -1.0f : 0.0f))
                                                 : fmax_cmp(fmin_cmp(av, 1.0f), -1.0f);
                    const float speed = __uint_as_float(jl[5]), power = __uint_as_float(jl[6]);
                    const float wa = sm[SC::BVEL + 4 * a + 2], wb = sm[SC::BVEL + 4 * b + 2];
                    const float arg = __fmaf_rn(-speed, A, wa - wb) * prm.motor_rho;
                    const float jr_ = power * tanh_spec(arg);
                    if ((jab >> 29) & 1u) sm[SC::BVEL + 4 * a + 2] = __fmaf_rn(-jr_, sm[SC::BII + a], wa);
                    if ((jab >> 30) & 1u) sm[SC::BVEL + 4 * b + 2] = __fmaf_rn(jr_, sm[SC::BII + b], wb);
                }
                g.sync();
            }
        }
        // thrusters in thruster order, by level in the same way
        if (SC::T > 0) {
            int tl = 0; uint32_t tp = 0u;
            const uint32_t *th = smu + SC::LVC_THR + 8 * (lane < SC::T ? lane : 0);
            if (lane < SC::T) { tp = th[0]; if ((tp >> 16) & 1u) tl = (tp >> 17) & 7u; }
            const int tmax = g.max_int(tl);
#pragma unroll 1
            for (int lvl = 1; lvl <= tmax; ++lvl) {
                if (tl == lvl) {
                    const int i = tp & 255;
                    const float tv = sm[SC::ACT + ((tp >> 8) & 255)];
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
        g.sync();       // boxes and velocities are final
        // joint pre-step (poses only; velocities are not read): the row goes to the env's scratch
        if (SC::J > 0 && lane < SC::J) {
            float4 q[6];
#pragma unroll
            for (int f = 0; f < 6; ++f) q[f] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            float accx = jacc0, accy = jacc1, accr = jacc2;
            if (!jon || !prm.warm_start) { accx = 0.0f; accy = 0.0f; accr = 0.0f; }
            int ang = 0;
            float kr = 0.0f, bias_r = 0.0f;
            if (jon) {
                const int a = jab & 255, b = (jab >> 8) & 255;
                float rax, ray, rbx, rby;
                rot2(sm[SC::BC + a], sm[SC::BS + a], __uint_as_float(jl[1]), __uint_as_float(jl[2]), rax, ray);
                rot2(sm[SC::BC + b], sm[SC::BS + b], __uint_as_float(jl[3]), __uint_as_float(jl[4]), rbx, rby);
                const float ma = sm[SC::BIM + a], mb = sm[SC::BIM + b], ia = sm[SC::BII + a], ib = sm[SC::BII + b];
                const float gx = (sm[SC::BPOS + 4 * b] + rbx) - (sm[SC::BPOS + 4 * a] + rax), gy = (sm[SC::BPOS + 4 * b + 1] + rby) - (sm[SC::BPOS + 4 * a + 1] + ray);
                const float msum = ma + mb;
                float k11 = msum; k11 = __fmaf_rn(ia * ray, ray, k11); k11 = __fmaf_rn(ib * rby, rby, k11);
                float k22 = msum; k22 = __fmaf_rn(ia * rax, rax, k22); k22 = __fmaf_rn(ib * rbx, rbx, k22);
                float k12 = -((ia * rax) * ray); k12 = __fmaf_rn(-(ib * rbx), rby, k12);
                const float det = __fmaf_rn(k11, k22, -(k12 * k12));
                const float inv_det = 1.0f / det;
                const float share = prm.joint_beta / msum;
                q[0] = make_float4(rax, ray, rbx, rby);
                q[1] = make_float4(k22 * inv_det, -(k12 * inv_det), k11 * inv_det, 0.0f);
                q[2] = make_float4(prm.joint_alpha * gx, prm.joint_alpha * gy, share * gx, share * gy);
                q[3] = make_float4(ma, mb, ia, ib);
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
            if (ang != 1) accr = 0.0f;
            q[1].w = __uint_as_float(jab);
            q[4] = make_float4(accx, accy, 0.0f, 0.0f);
            q[5] = make_float4(__int_as_float(ang), kr, bias_r, accr);
            float4 *jr = reinterpret_cast<float4 *>(scr + SC::SCR_JROW + kJointWords * lane);
#pragma unroll
            for (int f = 0; f < 6; ++f) jr[f] = q[f];
        }

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
                if (keep) surv()[nsurv + __popc(bal & g.lanes_below())] = (uint8_t)p;
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
        // the group's next env: its ticket has arrived by now; its meta head will have by the end of this env
        next_e = g.shflu(tn_raw, 0);
        if (next_e < (unsigned)prm.n_envs) next_head = load_meta_head(prm.state + (size_t)next_e * SC::ST_WORDS + SC::ST_META);

        // narrowphase: survivors of one kind at a time; pairs with an active manifold are staged in pair order, the
        // first G of them in shared memory, later ones in the staging area of the env's scratch
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
                    p = surv()[idx]; a = ptab[p] & 255; b = ptab[p] >> 8;
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
                    const int k = nrec + __popc(bal & g.lanes_below());
                    const uint32_t fa = smu[SC::BFL + a], fb = smu[SC::BFL + b];
                    const uint32_t ra = flag_role(fa), rb = flag_role(fb);
                    t_gb |= (ra == 1u && rb == 2u) || (ra == 2u && rb == 1u);
                    t_gr |= (ra == 1u && rb == 3u) || (ra == 3u && rb == 1u);
                    const uint32_t ab = (uint32_t)a | ((uint32_t)b << 5) | (act << 10) | ((uint32_t)p << 12) |
                                        (((fa & F_DYNAMIC) ? 1u : 0u) << 26) | (((fb & F_DYNAMIC) ? 1u : 0u) << 27);
                    const float nx = (act & 1u) ? m[0].nx : m[1].nx, ny = (act & 1u) ? m[0].ny : m[1].ny;
                    if (k < G) {
                        float *sg = sm + SC::STG + k;
                        sg[S_AB * G] = __uint_as_float(ab); sg[S_NX * G] = nx; sg[S_NY * G] = ny;
                        sg[S_PX0 * G] = m[0].px; sg[S_PY0 * G] = m[0].py; sg[S_PEN0 * G] = m[0].pen;
                        sg[S_PX1 * G] = m[1].px; sg[S_PY1 * G] = m[1].py; sg[S_PEN1 * G] = m[1].pen;
                    } else {
                        uint32_t *sg = scr + SC::SCR_STAGE + (size_t)k * kStageStride;
                        sg[S_AB] = ab; sg[S_NX] = __float_as_uint(nx); sg[S_NY] = __float_as_uint(ny);
                        sg[S_PX0] = __float_as_uint(m[0].px); sg[S_PY0] = __float_as_uint(m[0].py); sg[S_PEN0] = __float_as_uint(m[0].pen);
                        sg[S_PX1] = __float_as_uint(m[1].px); sg[S_PY1] = __float_as_uint(m[1].py); sg[S_PEN1] = __float_as_uint(m[1].pen);
                    }
                }
                nrec += __popc(bal);
            }
        }
        const bool touch_gb = g.any(t_gb), touch_gr = g.any(t_gr);
        g.sync();
        c_rec += (unsigned)nrec << 16;

        // Levels of the touching pairs (canonical order = staging order): one more than the highest level of an earlier pair
        // that shares a movable body.  Then every pair gets its row slot: rows are sorted by level, in staging order within
        // a level, and a byte table in the scratch says where each level starts.
        uint8_t *lstart = reinterpret_cast<uint8_t *>(scr + SC::SCR_LSTART);
        const bool crowded = nrec > G;      // more touching pairs than lanes: rare, handled by one lane through the scratch
        int cmax = 0, lvl = 0, slot = 0;
        uint32_t ab = 0u;
        if (!crowded) {
            const bool mine = lane < nrec;
            if (mine) ab = __float_as_uint(sm[SC::STG + S_AB * G + lane]);
            const int a = ab & 31, b = (ab >> 5) & 31;
            // every movable body collects the set of pairs that touch it; a pair's conflicts are the earlier members of its
            // bodies' sets; level r goes to the pairs whose conflicts all have a level already, round after round
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
#pragma unroll 1
            for (int r = 1; assigned != all; ++r) {
                const bool ready = mine && lvl == 0 && (conflicts & ~assigned) == 0u;
                if (ready) lvl = r;
                assigned |= g.ballot(ready);
            }
            cmax = g.max_int(lvl);
            int run = 0;
#pragma unroll 1
            for (int L = 1; L <= cmax; ++L) {
                const unsigned bal = g.ballot(lvl == L);
                if (lvl == L) slot = run + __popc(bal & g.lanes_below());
                if (lane == 0) lstart[L] = (uint8_t)run;
                run += __popc(bal);
            }
            if (lane == 0) lstart[cmax + 1] = (uint8_t)run;
        } else {
            // the pairs staged in shared memory join the others in the scratch
            {
                uint32_t *sg = scr + SC::SCR_STAGE + (size_t)lane * kStageStride;
#pragma unroll
                for (int f = 0; f < kStageWords; ++f) sg[f] = smu[SC::STG + f * G + lane];
            }
            g.sync();
            if (lane == 0) cmax = place_crowded_impl<SC>(scr, lstart, reinterpret_cast<uint8_t *>(smu + SC::SURV), nrec);
            g.sync();
            cmax = g.shfl(cmax, 0);
        }

        // rows: lane k of a round takes staged pair k, runs the pre-step of its active manifolds and writes the pair's row
        // into its slot; the accumulated impulses of the same pair in the previous step come from the lane that holds that
        // entry of the warm list (or from the state record beyond the lanes)
        int nman = 0;
        const ContactConsts cc = contact_consts();
#pragma unroll 1
        for (int base = 0; base < nrec; base += G) {
            const int k = base + lane;
            const bool mine = k < nrec;
            float nx = 0.0f, ny = 0.0f, pt[6] = { 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f };
            if (mine) {
                if (!crowded) {
                    const float *sg = sm + SC::STG + lane;
                    nx = sg[S_NX * G]; ny = sg[S_NY * G];
                    pt[0] = sg[S_PX0 * G]; pt[1] = sg[S_PY0 * G]; pt[2] = sg[S_PEN0 * G]; pt[3] = sg[S_PX1 * G]; pt[4] = sg[S_PY1 * G]; pt[5] = sg[S_PEN1 * G];
                } else {
                    const uint32_t *sg = scr + SC::SCR_STAGE + (size_t)k * kStageStride;
                    ab = __ldcg(sg + S_AB); nx = __uint_as_float(__ldcg(sg + S_NX)); ny = __uint_as_float(__ldcg(sg + S_NY));
                    pt[0] = __uint_as_float(__ldcg(sg + S_PX0)); pt[1] = __uint_as_float(__ldcg(sg + S_PY0)); pt[2] = __uint_as_float(__ldcg(sg + S_PEN0));
                    pt[3] = __uint_as_float(__ldcg(sg + S_PX1)); pt[4] = __uint_as_float(__ldcg(sg + S_PY1)); pt[5] = __uint_as_float(__ldcg(sg + S_PEN1));
                    slot = (int)__ldcg(sg + kStageWords);
                }
            } else ab = 0u;
            const unsigned amask = (ab >> 10) & 3u;
            const int p = (ab >> 12) & 127;
            // warm start values of this pair
            const int wi = mine ? (int)widx()[p] : 255;
            const int src = wi < G ? wi : 0;
            float4 w4 = make_float4(g.shflf(wacc.x, src), g.shflf(wacc.y, src), g.shflf(wacc.z, src), g.shflf(wacc.w, src));
            if (wi >= G && wi != 255) {
                const uint32_t *wr = st + SC::ST_WARM + kWarmWords * wi;
                w4 = make_float4(__uint_as_float(__ldcg(wr + 1)), __uint_as_float(__ldcg(wr + 2)), __uint_as_float(__ldcg(wr + 3)), __uint_as_float(__ldcg(wr + 4)));
            }
            if (wi == 255 || !prm.warm_start) w4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (!(amask & 1u)) { w4.x = 0.0f; w4.y = 0.0f; }
            if (!(amask & 2u)) { w4.z = 0.0f; w4.w = 0.0f; }
            nman += __popc(amask);
            if (mine) {
                const int a = ab & 31, b = (ab >> 5) & 31;
                const float ma = sm[SC::BIM + a], mb = sm[SC::BIM + b], ia = sm[SC::BII + a], ib = sm[SC::BII + b];
                const float fra = sm[SC::BFR + a], frb = sm[SC::BFR + b];
                const float mu = sqrtf(__fmaf_rn(fra, fra, frb * frb));
                const float er = fmin_cmp(sm[SC::BRE + a], sm[SC::BRE + b]);
                float4 *r = reinterpret_cast<float4 *>(scr + SC::SCR_ROWS + (size_t)slot * kRowWords);
                r[0] = make_float4(__uint_as_float(ab), nx, ny, mu);
                r[1] = make_float4(ma, mb, ia, ib);
#pragma unroll 1
                for (int mi = 0; mi < 2; ++mi) {
                    float rna = 0.0f, rnb = 0.0f, rta = 0.0f, rtb = 0.0f, massn = 0.0f, masst = 0.0f, target = 0.0f, corr = 0.0f;
                    if (amask & (1u << mi))
                        prestep_manifold<SC>(a, b, nx, ny, ma, mb, ia, ib, mi ? pt[3] : pt[0], mi ? pt[4] : pt[1], mi ? pt[5] : pt[2], er, sm, cc,
                                             rna, rnb, rta, rtb, massn, masst, target, corr);
                    r[2 + 2 * mi] = make_float4(rna, rnb, rta, rtb);
                    r[3 + 2 * mi] = make_float4(massn, masst, target, corr);
                }
                r[6] = w4;
            }
        }
        nman = g.sum_int(nman);
        c_man += (unsigned)nman | (1u << 16);
        // velocities (gravity, motors, thrusters) and this step's messages to the solve kernel
        for (int i = lane; i < SC::N; i += G)
            reinterpret_cast<float4 *>(st + SC::ST_VEL)[i] = reinterpret_cast<const float4 *>(sm + SC::BVEL)[i];
        if (lane == 0) {
            const uint32_t flags = (touch_gb ? 1u : 0u) | (touch_gr ? 2u : 0u) | (((gb >> 16) & 1u) << 2) | ((gb & 255u) << 8) | (((gb >> 8) & 255u) << 16) |
                                   ((uint32_t)cmax << 24);
            *reinterpret_cast<uint4 *>(st + SC::ST_META + META_NROWS) = make_uint4((uint32_t)nrec, flags, __float_as_uint(d0), active_mask | ((uint32_t)jmax << 16));
        }
    }
};


template <class SC, int G>
__global__ void __launch_bounds__(kBlockThreads, kMinBlocks) k2d_prep_kernel(const StepParams prm) {
    extern __shared__ __align__(16) uint32_t smem_raw[];
    constexpr int GPB = kBlockThreads / G;
    uint16_t *ptab = reinterpret_cast<uint16_t *>(smem_raw);
    for (int p = threadIdx.x; p < SC::NPAIRS; p += kBlockThreads) ptab[p] = pair_code<SC>(p);
    __syncthreads();
    const int gib = threadIdx.x / G;
    const int nslots = gridDim.x * GPB;
    uint32_t *region = smem_raw + SC::PTAB_WORDS + gib * region_words<SC, G>();
    Scene<SC, G> scene(region, ptab, prm);
    // Envs are handed out one at a time by a ticket counter: a group that is done takes the next one, so groups with
    // cheap scenes take more of them.  A group draws the ticket of its next env when it starts on an env and reads that
    // env's meta words half way through, so neither the counter nor the memory is waited for between envs.
    const Group<G> &g = scene.g;
    unsigned t = 0u;
    if (g.lane == 0) t = atomicAdd(prm.queue + Q_TICKET, 1u);
    t = g.shflu(t, 0);
    MetaHead head = { 0u, 0u, 0u };
    if (t < (unsigned)prm.n_envs) head = load_meta_head(prm.state + (size_t)t * SC::ST_WORDS + SC::ST_META);
    int taken = 0;
#pragma unroll 1
    while (t < (unsigned)prm.n_envs) {
        unsigned tn_raw = 0u, next_e = 0u;
        if (g.lane == 0) tn_raw = atomicAdd(prm.queue + Q_TICKET, 1u);
        MetaHead next_head = { 0u, 0u, 0u };
        if (head.status & 1u) {      // frozen env: nothing to prepare (the solve kernel reports done)
            next_e = g.shflu(tn_raw, 0);
            if (next_e < (unsigned)prm.n_envs) next_head = load_meta_head(prm.state + (size_t)next_e * SC::ST_WORDS + SC::ST_META);
        } else {
            scene.prepare((int)t, head, tn_raw, next_e, next_head);
        }
        g.sync();
        t = next_e; head = next_head;
        if ((++taken & 63) == 0) scene.flush();
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

// ================================================================ second half of a step: a group of kSolveLanes lanes per env
// The rows of a scene are copied to shared memory when its group starts (the first kRowCap pair rows and all joint rows;
// later pair rows, which few scenes have, are used where they are, in the scratch), so the sweeps below read and update
// them at shared-memory latency.  A row pointer is therefore a generic pointer.

// ---- angular row of a fixed joint or of a revolute joint beyond one of its limits (paper, "Fixed Joints",
// "Joint Limits"): j_r = (w_a - w_b + correction) / (1/I_a + 1/I_b), a loses j_r / I_a, b gains j_r / I_b.  A fixed
// joint's impulse is accumulated and warm-started; a limit only ever pushes back, applies no correction while the
// joint is already returning, and is not accumulated.  The row's last group: kind this step, inverse angular mass,
// correction, accumulated impulse.  Out of line: most joints are plain revolute joints.
template <int MODE>
__device__ __noinline__ float2 angular_row(float *jr, float ia, float ib, float wa, float wb) {
    const float4 ang4 = ld4(jr + JR_ANG);
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

// one visit of a joint row.  MODE 0: apply the accumulated impulses (warm start); 1: one solver iteration; 2: positional
// correction.  sv: the scene's bodies in shared memory (velocities; positions in mode 2).
template <int MODE>
__device__ __forceinline__ void solve_joint(float *jr, float4 *sv) {
    const float4 k4 = ld4(jr + JR_I11), mi4 = ld4(jr + JR_MA);
    const uint32_t jab = __float_as_uint(k4.w);
    const int a = jab & 255, b = (jab >> 8) & 255;
    const float ma = mi4.x, mb = mi4.y, ia = mi4.z, ib = mi4.w;
    if (MODE == 2) {
        const float cx = jr[JR_CX], cy = jr[JR_CY];
        if ((jab >> 29) & 1u) { float4 p = sv[a]; p.x = __fmaf_rn(ma, cx, p.x); p.y = __fmaf_rn(ma, cy, p.y); sv[a] = p; }
        if ((jab >> 30) & 1u) { float4 p = sv[b]; p.x = __fmaf_rn(-mb, cx, p.x); p.y = __fmaf_rn(-mb, cy, p.y); sv[b] = p; }
        return;
    }
    const float4 r4 = ld4(jr + JR_RAX);
    const float rax = r4.x, ray = r4.y, rbx = r4.z, rby = r4.w;
    const float4 va4 = sv[a], vb4 = sv[b];
    float vax = va4.x, vay = va4.y, wa = va4.z, vbx = vb4.x, vby = vb4.y, wb = vb4.z;
    const float2 acc = *reinterpret_cast<const float2 *>(jr + JR_ACCX);
    float lx, ly;
    if (MODE == 0) { lx = acc.x; ly = acc.y; }
    else {
        const float2 b2 = *reinterpret_cast<const float2 *>(jr + JR_BX);
        const float cx = __fmaf_rn(-wb, rby, vbx) - __fmaf_rn(-wa, ray, vax);
        const float cy = __fmaf_rn(wb, rbx, vby) - __fmaf_rn(wa, rax, vay);
        const float rx = -(cx + b2.x), ry = -(cy + b2.y);
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
    if ((jab >> 29) & 1u) sv[a] = make_float4(__fmaf_rn(-ma, lx, vax), __fmaf_rn(-ma, ly, vay), wa, 0.0f);
    if ((jab >> 30) & 1u) sv[b] = make_float4(__fmaf_rn(mb, lx, vbx), __fmaf_rn(mb, ly, vby), wb, 0.0f);
}

// one visit of a pair row (per active manifold the normal row, then the friction row), same modes
template <int MODE>
__device__ __forceinline__ void solve_pair(float *r, float4 *sv) {
    const float4 h0 = ld4(r + R_AB), h1 = ld4(r + R_MA);
    const uint32_t ab = __float_as_uint(h0.x);
    const int a = ab & 31, b = (ab >> 5) & 31;
    const unsigned amask = (ab >> 10) & 3u;
    const bool dyn_a = (ab >> 26) & 1u, dyn_b = (ab >> 27) & 1u;
    if (MODE == 2) {
        const float corr0 = r[R_M0 + M_CORR], corr1 = r[R_M1 + M_CORR];
        float4 pa = sv[a], pb = sv[b];
        if (amask & 1u) {
            const float ca = h1.x * corr0, cb = h1.y * corr0;
            pa.x = __fmaf_rn(-ca, h0.y, pa.x); pa.y = __fmaf_rn(-ca, h0.z, pa.y);
            pb.x = __fmaf_rn(cb, h0.y, pb.x); pb.y = __fmaf_rn(cb, h0.z, pb.y);
        }
        if (amask & 2u) {
            const float ca = h1.x * corr1, cb = h1.y * corr1;
            pa.x = __fmaf_rn(-ca, h0.y, pa.x); pa.y = __fmaf_rn(-ca, h0.z, pa.y);
            pb.x = __fmaf_rn(cb, h0.y, pb.x); pb.y = __fmaf_rn(cb, h0.z, pb.y);
        }
        if (dyn_a) sv[a] = pa;
        if (dyn_b) sv[b] = pb;
        return;
    }
    const float4 va4 = sv[a], vb4 = sv[b];
    float vax = va4.x, vay = va4.y, wa = va4.z, vbx = vb4.x, vby = vb4.y, wb = vb4.z;
    float4 acc = ld4(r + R_ACC);
    if (amask & 1u) {
        const float4 c0 = ld4(r + R_M0), c1 = ld4(r + R_M0 + 4);
        manifold_rows<MODE>(h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w, c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, acc.x, acc.y,
                            vax, vay, wa, vbx, vby, wb);
    }
    if (amask & 2u) {
        const float4 c0 = ld4(r + R_M1), c1 = ld4(r + R_M1 + 4);
        manifold_rows<MODE>(h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w, c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, acc.z, acc.w,
                            vax, vay, wa, vbx, vby, wb);
    }
    if (MODE == 1) *reinterpret_cast<float4 *>(r + R_ACC) = acc;
    if (dyn_a) sv[a] = make_float4(vax, vay, wa, 0.0f);
    if (dyn_b) sv[b] = make_float4(vbx, vby, wb, 0.0f);
}

constexpr int kRowCap = 12;   // pair rows of an env that are copied to shared memory for the solve; later rows are used in the scratch
constexpr int kLevCap = 32;   // level starts of an env kept in shared memory; a scene with more levels reads the table in its scratch

// n groups of 16 bytes from memory to shared memory by the GS lanes of a group, B per lane in flight at a time
template <int B, int GS>
__device__ __forceinline__ void stage_groups(float4 *dst, const float4 *src, int n, int lane) {
#pragma unroll 1
    for (int base = 0; base < n; base += B * GS) {
        float4 v[B];
#pragma unroll
        for (int k = 0; k < B; ++k) { const int i = base + lane + k * GS; v[k] = (i < n) ? __ldcg(src + i) : make_float4(0.0f, 0.0f, 0.0f, 0.0f); }
#pragma unroll
        for (int k = 0; k < B; ++k) { const int i = base + lane + k * GS; if (i < n) dst[i] = v[k]; }
    }
}

template <class SC>
__global__ void __launch_bounds__(kSolveThreads) k2d_solve_kernel(const StepParams prm) {
    constexpr int GS = kSolveLanes, SPB = kSolveThreads / GS;     // lanes per scene, scenes per block
    constexpr int JPL = (SC::J + GS - 1) / GS;                    // joints a lane may own: lane, lane + GS, ...
    // per scene: the bodies' velocities (later positions), the joint rows, the first kRowCap pair rows, the first row of every level
    constexpr int S_BODY = 0, S_JROW = 4 * SC::N, S_ROWS = S_JROW + kJointWords * SC::J, S_LSTART = S_ROWS + kRowWords * kRowCap;
    constexpr int S_WORDS = S_LSTART + kLevCap / 4;
    __shared__ __align__(16) float s_scene[SPB * S_WORDS];
    const Group<GS> g;
    const int lane = g.lane, sb = threadIdx.x / GS;
    const int e = blockIdx.x * SPB + sb;
    const bool in_range = e < prm.n_envs;
    uint32_t *st = prm.state + (size_t)(in_range ? e : 0) * SC::ST_WORDS;
    float *stf = reinterpret_cast<float *>(st);
    uint4 m0 = make_uint4(0u, 0u, 0u, 0u), m1 = m0;
    if (in_range) { m0 = *reinterpret_cast<const uint4 *>(st + SC::ST_META); m1 = *reinterpret_cast<const uint4 *>(st + SC::ST_META + 4); }
    // frozen env: reports done, nothing else
    const bool frozen = in_range && (m0.w & 1u);
    if (frozen && lane == 0) { prm.reward[e] = 0.0f; prm.done[e] = 1; }
    const bool live = in_range && !frozen;
    const unsigned wmask = __ballot_sync(0xffffffffu, live);      // the warp's lanes that go on: its groups stay in step level by level
    if (!live) return;
    float *ss = s_scene + sb * S_WORDS;
    float4 *sv = reinterpret_cast<float4 *>(ss + S_BODY);
    float *sj = ss + S_JROW, *sr = ss + S_ROWS;
    uint8_t *sl = reinterpret_cast<uint8_t *>(ss + S_LSTART);
    uint32_t *scr = prm.scratch + (size_t)e * SC::SCRATCH_WORDS;
    float *rows = reinterpret_cast<float *>(scr + SC::SCR_ROWS);
    const uint8_t *lstart = reinterpret_cast<const uint8_t *>(scr + SC::SCR_LSTART);
    const int nrows = (int)m1.x;
    const uint32_t flags = m1.y, active = m1.w & 0xffffu;
    const int cmax = (int)(flags >> 24), jmax = (int)((m1.w >> 16) & 15u);
    const int cmax_w = __reduce_max_sync(wmask, cmax), jmax_w = __reduce_max_sync(wmask, jmax);
    // velocities, joint rows, level starts, pair rows -> shared memory
    {
        constexpr int NB = SC::N + 6 * SC::J;       // the velocities and the joint rows are contiguous neither in memory nor here: two sources, one volley
        constexpr int KB = (NB + GS - 1) / GS;
        float4 v[KB];
        uint32_t lw = 0u;
        const float4 *src_v = reinterpret_cast<const float4 *>(stf + SC::ST_VEL), *src_j = reinterpret_cast<const float4 *>(scr + SC::SCR_JROW);
#pragma unroll
        for (int k = 0; k < KB; ++k) {
            const int i = lane + k * GS;
            v[k] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (i < SC::N) v[k] = __ldcg(src_v + i); else if (i < NB) v[k] = __ldcg(src_j + (i - SC::N));
        }
        static_assert(kLevCap / 4 <= 2 * GS, "level starts: at most two words per lane");
        uint32_t lw2 = 0u;
        if (lane < kLevCap / 4) lw = __ldcg(scr + SC::SCR_LSTART + lane);
        if (lane + GS < kLevCap / 4) lw2 = __ldcg(scr + SC::SCR_LSTART + lane + GS);
#pragma unroll
        for (int k = 0; k < KB; ++k) {
            const int i = lane + k * GS;
            if (i < SC::N) sv[i] = v[k]; else if (i < NB) reinterpret_cast<float4 *>(sj)[i - SC::N] = v[k];
        }
        if (lane < kLevCap / 4) reinterpret_cast<uint32_t *>(sl)[lane] = lw;
        if (lane + GS < kLevCap / 4) reinterpret_cast<uint32_t *>(sl)[lane + GS] = lw2;
    }
    stage_groups<6, GS>(reinterpret_cast<float4 *>(sr), reinterpret_cast<const float4 *>(rows), 7 * (nrows < kRowCap ? nrows : kRowCap), lane);
    g.sync();
    // this lane's joints and their levels (0: the joint takes no part)
    int jlev[JPL > 0 ? JPL : 1];
#pragma unroll
    for (int q = 0; q < JPL; ++q) {
        const int j = lane + q * GS;
        jlev[q] = 0;
        if (j < SC::J) {
            const uint32_t jab = __float_as_uint(sj[j * kJointWords + JR_JAB]);
            if ((jab >> 24) & 1u) jlev[q] = (int)((jab >> 25) & 7u);
        }
    }
#define K2D_ROW(r) ((r) < kRowCap ? sr + (r) * kRowWords : rows + (r) * kRowWords)
#define K2D_LSTART(L) ((L) < kLevCap ? (int)sl[L] : (int)lstart[L])
    // One sweep over the pair rows / the joint rows, level by level; the rows of a level go to the lanes round robin.  All
    // groups of the warp walk the same number of levels and meet after each, so that they execute the rows together.
#define K2D_SWEEP_PAIRS(MODE)                                                                         \
    _Pragma("unroll 1") for (int L = 1; L <= cmax_w; ++L) {                                           \
        int r = 0, r1 = 0;                                                                            \
        if (L <= cmax) { r = K2D_LSTART(L); r1 = K2D_LSTART(L + 1); }                                 \
        const int rounds = (__reduce_max_sync(wmask, r1 - r) + GS - 1) / GS;                          \
        r += lane;                                                                                    \
        _Pragma("unroll 1") for (int q = 0; q < rounds; ++q, r += GS)                                 \
            if (r < r1) solve_pair<MODE>(K2D_ROW(r), sv);                                             \
        __syncwarp(wmask);                                                                            \
    }
#define K2D_SWEEP_JOINTS(MODE)                                                                        \
    if (SC::J > 0) {                                                                                  \
        _Pragma("unroll 1") for (int L = 1; L <= jmax_w; ++L) {                                       \
            _Pragma("unroll") for (int q = 0; q < JPL; ++q)                                           \
                if (jlev[q] == L) solve_joint<MODE>(sj + (lane + q * GS) * kJointWords, sv);          \
            __syncwarp(wmask);                                                                        \
        }                                                                                             \
    }
    // warm start: contacts, then joints (Algorithm 1); solver iterations: joints, then contacts
    K2D_SWEEP_PAIRS(0)
    K2D_SWEEP_JOINTS(0)
#pragma unroll 1
    for (int it = 0; it < prm.solver_iters; ++it) {
        K2D_SWEEP_JOINTS(1)
        K2D_SWEEP_PAIRS(1)
    }
    // Euler step with the solved velocities; the velocities go back to the state record and the array holds positions from here on
    bool finite = true;
    {
        constexpr int KN = (SC::N + GS - 1) / GS;
        float4 p[KN];
#pragma unroll
        for (int k = 0; k < KN; ++k) { const int i = lane + k * GS; p[k] = (i < SC::N) ? ld4(stf + SC::ST_POS + 4 * i) : make_float4(0.0f, 0.0f, 0.0f, 0.0f); }
#pragma unroll
        for (int k = 0; k < KN; ++k) {
            const int i = lane + k * GS;
            if (i < SC::N) {
                const float4 v4 = sv[i];
                float4 p4 = p[k];
                if ((active >> i) & 1u) { p4.x = __fmaf_rn(prm.dt, v4.x, p4.x); p4.y = __fmaf_rn(prm.dt, v4.y, p4.y); p4.z = __fmaf_rn(prm.dt, v4.z, p4.z); }
                finite = finite && finite_bits(v4.x) && finite_bits(v4.y) && finite_bits(v4.z);
                st4(stf + SC::ST_VEL + 4 * i, v4.x, v4.y, v4.z);
                sv[i] = p4;
            }
        }
    }
    __syncwarp(wmask);
    // positional corrections: every active manifold moves its two bodies apart along the normal, then the joints close their gaps
    K2D_SWEEP_PAIRS(2)
    K2D_SWEEP_JOINTS(2)
    for (int i = lane; i < SC::N; i += GS) {
        const float4 p4 = sv[i];
        finite = finite && finite_bits(p4.x) && finite_bits(p4.y) && finite_bits(p4.z);
        st4(stf + SC::ST_POS + 4 * i, p4.x, p4.y, p4.z);
    }
    finite = !g.any(!finite);
    // reward and termination (paper, "Reward"): green touches blue = +1, green touches red = -1, either ends the episode
    const int step_count = (int)m0.x + 1;
    const bool touch_gb = (flags & 1u) != 0u, touch_gr = (flags & 2u) != 0u;
    const bool timeout = prm.max_episode_steps > 0 && step_count >= prm.max_episode_steps;
    float reward = (float)((int)touch_gb - (int)touch_gr);
    if (prm.dense_kappa != 0.0f && ((flags >> 2) & 1u)) {
        const float4 pg = sv[(flags >> 8) & 255u], pb = sv[(flags >> 16) & 255u];
        const float dx = pb.x - pg.x, dy = pb.y - pg.y;
        reward = reward + prm.dense_kappa * (__uint_as_float(m1.z) - sqrtf(dot2(dx, dy, dx, dy)));
    }
    bool done = touch_gb || touch_gr || timeout;
    uint32_t status = m0.w;
    if (!finite) { reward = 0.0f; done = true; status |= 1u; }
    if (lane == 0) {
        prm.reward[e] = reward;
        prm.done[e] = done ? 1 : 0;
        if (!finite) atomicAdd(prm.counters + 0, 1ULL);
    }
    if (!(done && prm.auto_reset != 0)) {
        // the accumulated impulses of this step's rows warm-start the next step
        for (int r = lane; r < nrows; r += GS) {
            const float *row = K2D_ROW(r);
            const float4 acc = ld4(row + R_ACC);
            uint32_t *wr = st + SC::ST_WARM + kWarmWords * r;
            wr[0] = (__float_as_uint(row[R_AB]) >> 12) & 127u;
            wr[1] = __float_as_uint(acc.x); wr[2] = __float_as_uint(acc.y); wr[3] = __float_as_uint(acc.z); wr[4] = __float_as_uint(acc.w);
        }
        for (int j = lane; j < SC::J; j += GS) {
            const float *jr = sj + j * kJointWords;
            st[SC::ST_JACC + 3 * j] = __float_as_uint(jr[JR_ACCX]);
            st[SC::ST_JACC + 3 * j + 1] = __float_as_uint(jr[JR_ACCY]);
            st[SC::ST_JACC + 3 * j + 2] = __float_as_uint(jr[JR_ACCR]);
        }
        if (lane == 0) {
            st[SC::ST_META + META_STEP] = (uint32_t)step_count;
            st[SC::ST_META + META_STATUS] = status;
        }
        return;
    }
#undef K2D_SWEEP_JOINTS
#undef K2D_SWEEP_PAIRS
#undef K2D_LSTART
#undef K2D_ROW
    // auto-reset of a finished env: next level (its own, or drawn from the pool by the hash of seed, global env index
    // and episode), pose from the level, no accumulated impulses
    const int episode = (int)m0.y + 1;
    int level = (int)m0.z;
    if (prm.auto_reset == 2) {
        const unsigned long long h = mix64(prm.seed + ((unsigned long long)(prm.env_offset + e) + 1ULL) * 0x9E3779B97F4A7C15ULL +
                                           (unsigned long long)episode * 0xD1B54A32D192ED03ULL);
        level = (int)(h % (unsigned long long)prm.n_levels);
    }
    const float *lv = reinterpret_cast<const float *>(prm.levels + (size_t)level * SC::LV_WORDS);
    for (int i = lane; i < SC::N; i += GS) {
        st4(stf + SC::ST_POS + 4 * i, lv[SC::LV_X + i], lv[SC::LV_Y + i], lv[SC::LV_TH + i]);
        st4(stf + SC::ST_VEL + 4 * i, lv[SC::LV_VX + i], lv[SC::LV_VY + i], lv[SC::LV_W + i]);
    }
    for (int j = lane; j < 3 * SC::J; j += GS) st[SC::ST_JACC + j] = 0u;
    if (lane == 0) {
        *reinterpret_cast<uint4 *>(st + SC::ST_META) = make_uint4(0u, (uint32_t)episode, (uint32_t)level, 0u);
        st[SC::ST_META + META_NROWS] = 0u;
        atomicAdd(prm.counters + 1, 1ULL);
    }
}

// ---------------------------------------------------------------- reset kernel: one block per env
template <class SC>
__global__ void k2d_reset_kernel(uint32_t *state, const uint32_t *levels, const int *level_ids, int n_envs, int n_levels) {
    const int e = blockIdx.x;
    if (e >= n_envs) return;
    const int l = level_ids ? level_ids[e] : e % n_levels;
    uint32_t *st = state + (size_t)e * SC::ST_WORDS;
    const uint32_t *lv = levels + (size_t)l * SC::LV_WORDS;
    for (int i = threadIdx.x; i < SC::ST_WARM; i += blockDim.x) {
        uint32_t v = 0u;
        if (i < 8 * SC::N) {
            const int half = i / (4 * SC::N), r = i - half * 4 * SC::N, body = r >> 2, f = r & 3;     // position or velocity group, body, component
            if (f < 3) v = lv[SC::LV_X + (3 * half + f) * SC::N + body];
        } else if (i == SC::ST_META + META_LEVEL) v = (uint32_t)l;
        st[i] = v;
    }
}

// ---------------------------------------------------------------- observation kernel: one warp per env
// Each lane writes whole entity rows (a shape, one side of a joint, a thruster) into the warp's
// shared-memory image of the observation, then the warp copies the image out with coalesced stores.
template <class SC>
__global__ void __launch_bounds__(kObsThreads) k2d_obs_kernel(const uint32_t *state, const uint32_t *levels, float *obs,
                                                              int n_envs, int n_actions, int n_polygons, int n_circles,
                                                              int n_joints, int n_thrusters) {
    extern __shared__ __align__(16) float obs_smem[];
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int e = blockIdx.x * (kObsThreads / 32) + w;
    if (e >= n_envs) return;
    const int n_shapes = n_polygons + n_circles;
    const int jw = 11 + n_actions;
    const int width = n_shapes * 29 + 2 * n_joints * jw + 6 * n_thrusters;
    float *img = obs_smem + (size_t)w * ((width + 2 * SC::N + 3) / 4 * 4);
    float *cs = img + width;                 // cos, sin of every shape's angle
    const uint32_t *st = state + (size_t)e * SC::ST_WORDS;
    const uint32_t *lv = levels + (size_t)st[SC::ST_META + META_LEVEL] * SC::LV_WORDS;
    const float *stf = reinterpret_cast<const float *>(st);
    const float *lvf = reinterpret_cast<const float *>(lv);
    for (int ci = lane; ci < n_shapes; ci += 32) {
        const int i = ci < n_polygons ? ci : SC::P + (ci - n_polygons);     // internal shape index
        float c, sn;
        sincos_spec(stf[SC::ST_POS + 4 * i + 2], c, sn);
        cs[i] = c; cs[SC::N + i] = sn;
        float *o = img + ci * 29;
        const uint32_t fl = lv[SC::LV_FLAGS + i];
        if (!(fl & F_ACTIVE)) {
            for (int f = 0; f < 29; ++f) o[f] = 0.0f;
            continue;
        }
        const int nv = flag_nverts(fl);
        const uint32_t role = flag_role(fl);
        const bool poly = i < SC::P;
        o[0] = stf[SC::ST_POS + 4 * i]; o[1] = stf[SC::ST_POS + 4 * i + 1]; o[2] = stf[SC::ST_VEL + 4 * i]; o[3] = stf[SC::ST_VEL + 4 * i + 1];
        o[4] = lvf[SC::LV_IM + i]; o[5] = lvf[SC::LV_II + i]; o[6] = lvf[SC::LV_DENS + i];
        o[7] = tanh_spec(stf[SC::ST_VEL + 4 * i + 2] * 0.1f);
#pragma unroll
        for (int r = 0; r < 4; ++r) o[8 + r] = (role == (uint32_t)r) ? 1.0f : 0.0f;
        o[12] = sn; o[13] = c; o[14] = lvf[SC::LV_FR + i]; o[15] = lvf[SC::LV_RE + i];
        o[16] = poly ? 1.0f : 0.0f; o[17] = poly ? 0.0f : 1.0f;
        o[18] = poly ? 0.0f : lvf[SC::LV_RAD + (poly ? 0 : i - SC::P)];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool on = poly && k < nv;
            o[19 + 2 * k] = on ? lvf[SC::LV_PVX + 4 * (poly ? i : 0) + k] : 0.0f;
            o[20 + 2 * k] = on ? lvf[SC::LV_PVY + 4 * (poly ? i : 0) + k] : 0.0f;
        }
        o[27] = (poly && nv == 3) ? 1.0f : 0.0f;
        o[28] = (poly && nv != 3) ? 1.0f : 0.0f;
    }
    __syncwarp();
    float *jrows = img + n_shapes * 29;
    for (int row = lane; row < 2 * n_joints; row += 32) {
        const int j = row >> 1, d = row & 1;
        const uint32_t *jl = lv + SC::LV_JOINT + kJointLevelWords * j;
        const uint32_t jab = jl[0];
        float *o = jrows + row * jw;
        for (int f = 0; f < jw; ++f) o[f] = 0.0f;
        if ((jab >> 28) & 1u) {
            const int a = jab & 255, b = (jab >> 8) & 255;
            const int from = d ? b : a, to = d ? a : b;
            o[0] = 1.0f; o[1] = (jl[10] & 1u) ? 1.0f : 0.0f;
#pragma unroll
            for (int f = 2; f < 6; ++f) { const int side = ((f - 2) >> 1) ^ d; o[f] = __uint_as_float(jl[1 + 2 * side + ((f - 2) & 1)]); }
            o[6] = __uint_as_float(jl[6]); o[7] = __uint_as_float(jl[5]);
            const int bind = (int)((jab >> 16) & 255);
            if (bind < n_actions) o[9 + bind] = 1.0f;
            o[9 + n_actions] = __fmaf_rn(cs[SC::N + to], cs[from], -(cs[to] * cs[SC::N + from]));
            o[10 + n_actions] = __fmaf_rn(cs[to], cs[from], cs[SC::N + to] * cs[SC::N + from]);
        }
    }
    float *trows = jrows + 2 * n_joints * jw;
    for (int t = lane; t < n_thrusters; t += 32) {
        const uint32_t *th = lv + SC::LV_THR + 8 * t;
        const uint32_t tp = th[0];
        float *o = trows + t * 6;
        for (int f = 0; f < 6; ++f) o[f] = 0.0f;
        if ((tp >> 20) & 1u) {
            const int i = tp & 255;
            float dx, dy;
            rot2(cs[i], cs[SC::N + i], __uint_as_float(th[3]), __uint_as_float(th[4]), dx, dy);
            o[0] = 1.0f; o[1] = __uint_as_float(th[1]); o[2] = __uint_as_float(th[2]); o[3] = __uint_as_float(th[5]);
            o[4] = dy; o[5] = dx;
        }
    }
    __syncwarp();
    float *out = obs + (size_t)e * width;
    if (((width & 3) == 0) && ((reinterpret_cast<uintptr_t>(obs) & 15) == 0)) {
        const float4 *src = reinterpret_cast<const float4 *>(img);
        float4 *dst = reinterpret_cast<float4 *>(out);
        for (int q = lane; q < width / 4; q += 32) dst[q] = src[q];
    } else {
        for (int q = lane; q < width; q += 32) out[q] = img[q];
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
            const float x = stf[SC::ST_POS + 4 * i], y = stf[SC::ST_POS + 4 * i + 1];
            const uint32_t role = flag_role(fl);
            uint32_t rgb = role == 1u ? (200u << 8) : role == 2u ? (220u << 16) : role == 3u ? 220u : ((fl & F_DYNAMIC) ? 0x808080u : 0x404040u);
            s_col[i] = rgb | 0xff000000u;
            if (i < SC::P) {
                nv = (int)flag_nverts(fl);
                float c, sn;
                sincos_spec(stf[SC::ST_POS + 4 * i + 2], c, sn);
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
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t *img = pixels + (size_t)e * kPix * kPix;
    // a warp paints one row at a time in registers: lane l holds the pixels of columns l, l + 32, l + 64, l + 96;
    // the shapes whose box reaches the row go over it in index order, each only over the 32-column blocks its box
    // touches, so the highest index ends up on top
    for (int r = warp; r < kPix; r += kRenderThreads / 32) {
        const float py = 5.75f - ((float)r + 0.5f) * 0.05f;
        bool reach = false;
        if (lane < SC::N && s_nv[lane] >= 0) reach = s_rng[lane].z <= r && r <= s_rng[lane].w;
        unsigned m = __ballot_sync(0xffffffffu, reach);
        uint32_t col[4] = { 0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu };
        while (m) {
            const int i = __ffs(m) - 1;
            m &= m - 1u;
            const int4 rng = s_rng[i];
            const int nv = s_nv[i];
            const float4 nx = s_nx[i], ny = s_ny[i], off = s_off[i];
            const uint32_t shape_col = s_col[i];
            // the row's share of every face's dot product (polygon) or of the squared distance (circle)
            const float t0 = ny.x * py, t1 = ny.y * py, t2 = ny.z * py, t3 = ny.w * py;
            const float dy = py - ny.x, dy2 = dy * dy;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (rng.y < 32 * k || rng.x > 32 * k + 31) continue;       // the same for the whole warp
                const float px = -3.125f + ((float)(32 * k + lane) + 0.5f) * 0.05f;
                bool inside;
                if (nv > 0) {
                    inside = !(__fmaf_rn(nx.x, px, t0) - off.x > 0.0f) && !(__fmaf_rn(nx.y, px, t1) - off.y > 0.0f) &&
                             !(__fmaf_rn(nx.z, px, t2) - off.z > 0.0f) && (nv < 4 || !(__fmaf_rn(nx.w, px, t3) - off.w > 0.0f));
                } else {
                    const float dx = px - nx.x;
                    inside = __fmaf_rn(dx, dx, dy2) <= off.x;
                }
                if (inside) col[k] = shape_col;
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (32 * k + lane < kPix) img[r * kPix + 32 * k + lane] = col[k];
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

}  // namespace k2d
