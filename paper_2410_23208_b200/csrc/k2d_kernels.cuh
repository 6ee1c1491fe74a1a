// k2d_kernels.cuh -- device code of the batched 2D rigid-body environment step (sm_100a).
//
// One group of G lanes (G = 32: one warp; 16 or 8: two or four scenes per warp) owns one scene.
// The scene's state is loaded from HBM once per launch, kept in shared memory across all fused
// steps, and written back once.  Within a step the lanes of the group work on bodies, polygon
// vertices, shape pairs (bounding-box test, narrowphase, contact pre-step) and constraint rows.
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

constexpr int kBlockThreads = 128;
constexpr int kMaxActions = 16;
constexpr int kRecWords = 24;   // contact pair record
constexpr int kWarmWords = 5;   // pair index + 4 accumulated impulses

// ---------------------------------------------------------------- size classes and layouts
template <int P_, int C_, int J_, int T_, int CAP_>
struct SizeClass {
    static constexpr int P = P_, C = C_, N = P_ + C_, J = J_, T = T_;
    static constexpr int NPP = P * (P - 1) / 2, NPC = P * C, NCC = C * (C - 1) / 2;
    static constexpr int NPAIRS = NPP + NPC + NCC, NSLOTS = 2 * NPP + NPC + NCC;
    static constexpr int CAP = CAP_ < NPAIRS ? CAP_ : NPAIRS;   // pair records kept in shared memory
    static constexpr int OVF = NPAIRS - CAP;                     // the rest live in global scratch
    static constexpr int MASKW = (NPAIRS + 31) / 32;
    static constexpr int P4 = 4 * P;
    // level record (32-bit words)
    static constexpr int LV_X = 0, LV_Y = N, LV_TH = 2 * N, LV_VX = 3 * N, LV_VY = 4 * N, LV_W = 5 * N;
    static constexpr int LV_IM = 6 * N, LV_II = 7 * N, LV_FR = 8 * N, LV_RE = 9 * N, LV_FLAGS = 10 * N, LV_DENS = 11 * N;
    static constexpr int LV_RAD = 12 * N;
    static constexpr int LV_PVX = LV_RAD + C, LV_PVY = LV_PVX + P4, LV_PNX = LV_PVY + P4, LV_PNY = LV_PNX + P4, LV_ELEN = LV_PNY + P4;
    static constexpr int LV_JOINT = LV_ELEN + P4;        // J x 8: packed, anchor a xy, anchor b xy, speed, power, pad
    static constexpr int LV_THR = LV_JOINT + 8 * J;      // T x 8: packed, pos xy, dir xy, power, pad, pad
    static constexpr int LV_MASK = LV_THR + 8 * T;
    static constexpr int LV_WORDS = (LV_MASK + MASKW + 3) / 4 * 4;
    // state record: bodies (same order as shared memory), joint impulses, meta, warm list
    static constexpr int ST_BODY = 0, ST_JACC = 6 * N, ST_META = ST_JACC + 2 * J, ST_WARM = ST_META + 8;
    static constexpr int ST_WORDS = (ST_WARM + kWarmWords * NPAIRS + 3) / 4 * 4;
    static constexpr int SCRATCH_WORDS = OVF * (kRecWords + kWarmWords);
    // shared memory region of one scene (words)
    static constexpr int BX = 0, BY = N, BTH = 2 * N, BVX = 3 * N, BVY = 4 * N, BW = 5 * N;
    static constexpr int BIM = 6 * N, BII = 7 * N, BFR = 8 * N, BRE = 9 * N, BC = 10 * N, BS = 11 * N, BFL = 12 * N;
    static constexpr int RAD = 13 * N;
    static constexpr int WVX = RAD + C, WVY = WVX + P4, WNX = WVY + P4, WNY = WNX + P4, WOFF = WNY + P4, ELEN = WOFF + P4;
    static constexpr int AMINX = ELEN + P4, AMINY = AMINX + N, AMAXX = AMINY + N, AMAXY = AMAXX + N;
    static constexpr int JNT = AMAXY + N;                // 14 arrays of J
    static constexpr int MASK = JNT + 14 * J;
    static constexpr int ACT = MASK + MASKW;
    static constexpr int SURV = ACT + kMaxActions;       // bytes
    static constexpr int WIDX = SURV + (NPAIRS + 3) / 4; // bytes
    static constexpr int REC = WIDX + (NPAIRS + 3) / 4;
    static constexpr int WARM = REC + kRecWords * CAP;
    static constexpr int REGION_RAW = WARM + kWarmWords * CAP;
    static constexpr int PTAB_WORDS = (NPAIRS + 1) / 2;  // block-shared pair table, 16 bits per pair
};
// joint arrays inside JNT
enum { JA_AB = 0, JA_RAX, JA_RAY, JA_RBX, JA_RBY, JA_I11, JA_I12, JA_I22, JA_BX, JA_BY, JA_CX, JA_CY, JA_ACCX, JA_ACCY };
// record fields
enum { R_AB = 0, R_NX, R_NY, R_MU, R_M0 = 4 };
enum { M_RNA = 0, M_RNB, M_RTA, M_RTB, M_MASSN, M_MASST, M_TARGET, M_CORR, M_ACCN, M_ACCT, M_WORDS };
static_assert(R_M0 + 2 * M_WORDS == kRecWords, "record size");

// shared-memory words per scene: padded so that the groups of one warp start in different banks
template <class SC, int G>
__host__ __device__ constexpr int region_words() { return (SC::REGION_RAW + 31) / 32 * 32 + (G < 32 ? G : 0); }

// body flag word
constexpr uint32_t F_ACTIVE = 1u, F_DYNAMIC = 2u;
__host__ __device__ inline uint32_t flag_role(uint32_t f) { return (f >> 2) & 3u; }
__host__ __device__ inline uint32_t flag_nverts(uint32_t f) { return (f >> 4) & 7u; }
// joint packed word: a | b<<8 | binding<<16 | on<<24 | level<<25 | active<<28
// thruster packed word: shape | binding<<8 | on<<16 | level<<17 | active<<20
// record AB word: a | b<<5 | amask<<10 | pair<<12 | level<<19 | dynA<<26 | dynB<<27

struct StepParams {
    uint32_t *state;
    const uint32_t *levels;
    const float *actions;
    float *reward;
    uint8_t *done;
    unsigned long long *counters;
    uint32_t *scratch;
    float *trace;
    int n_envs, n_steps, n_actions, n_levels;
    int solver_iters, warm_start, auto_reset, max_episode_steps;
    float dt, gdt, contact_alpha, contact_beta, slop, rest_thr, face_tol, joint_alpha, joint_beta, motor_rho, aabb_margin;
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
    __device__ __forceinline__ int max_int(int v) const { return __reduce_max_sync(mask, v); }
    __device__ __forceinline__ bool any(bool p) const { return __ballot_sync(mask, p) != 0; }
    __device__ __forceinline__ unsigned lanes_below() const { return (1u << lane) - 1u; }
};

// one manifold as the narrowphase leaves it
struct Manifold { float px, py, nx, ny, pen; };

// ---------------------------------------------------------------- scene processing
template <class SC, int G>
struct Scene {
    float *sm;            // this scene's shared-memory region
    uint32_t *smu;
    const uint16_t *ptab; // block-shared pair table
    uint32_t *ovf;        // this group's overflow scratch in global memory (SC::OVF > 0 only)
    const StepParams &prm;
    Group<G> g;
    int lane;

    __device__ __forceinline__ Scene(uint32_t *region, const uint16_t *pt, uint32_t *scratch, const StepParams &p)
        : sm(reinterpret_cast<float *>(region)), smu(region), ptab(pt), ovf(scratch), prm(p), g() { lane = g.lane; }

    __device__ __forceinline__ uint8_t *surv() { return reinterpret_cast<uint8_t *>(smu + SC::SURV); }
    __device__ __forceinline__ uint8_t *widx() { return reinterpret_cast<uint8_t *>(smu + SC::WIDX); }

    // record / warm accessors; k >= CAP lives in global scratch
    __device__ __forceinline__ float rec_ld(int f, int k) const {
        if (SC::OVF == 0 || k < SC::CAP) return sm[SC::REC + f * SC::CAP + k];
        return __uint_as_float(ovf[(k - SC::CAP) * kRecWords + f]);
    }
    __device__ __forceinline__ void rec_st(int f, int k, float v) {
        if (SC::OVF == 0 || k < SC::CAP) sm[SC::REC + f * SC::CAP + k] = v;
        else ovf[(k - SC::CAP) * kRecWords + f] = __float_as_uint(v);
    }
    __device__ __forceinline__ uint32_t warm_ld(int f, int k) const {
        if (SC::OVF == 0 || k < SC::CAP) return smu[SC::WARM + f * SC::CAP + k];
        return ovf[SC::OVF * kRecWords + (k - SC::CAP) * kWarmWords + f];
    }
    __device__ __forceinline__ void warm_st(int f, int k, uint32_t v) {
        if (SC::OVF == 0 || k < SC::CAP) smu[SC::WARM + f * SC::CAP + k] = v;
        else ovf[SC::OVF * kRecWords + (k - SC::CAP) * kWarmWords + f] = v;
    }

    // ---- level constants into shared memory
    __device__ void load_level_consts(const uint32_t *lv) {
        for (int i = lane; i < SC::N; i += G) {
            smu[SC::BIM + i] = lv[SC::LV_IM + i];
            smu[SC::BII + i] = lv[SC::LV_II + i];
            smu[SC::BFR + i] = lv[SC::LV_FR + i];
            smu[SC::BRE + i] = lv[SC::LV_RE + i];
            smu[SC::BFL + i] = lv[SC::LV_FLAGS + i];
        }
        for (int i = lane; i < SC::C; i += G) smu[SC::RAD + i] = lv[SC::LV_RAD + i];
        for (int i = lane; i < SC::P4; i += G) smu[SC::ELEN + i] = lv[SC::LV_ELEN + i];
        for (int i = lane; i < SC::MASKW; i += G) smu[SC::MASK + i] = lv[SC::LV_MASK + i];
    }
    __device__ void load_level_pose(const uint32_t *lv) {
        for (int i = lane; i < 6 * SC::N; i += G) smu[SC::BX + i] = lv[SC::LV_X + i];
        for (int i = lane; i < SC::J; i += G) { sm[SC::JNT + JA_ACCX * SC::J + i] = 0.0f; sm[SC::JNT + JA_ACCY * SC::J + i] = 0.0f; }
        for (int i = lane; i < (SC::NPAIRS + 3) / 4; i += G) smu[SC::WIDX + i] = 0xffffffffu;
    }

    // ---- narrowphase: polygon a against polygon b (world data in shared memory)
    __device__ __forceinline__ void max_separation(int x, int cntx, const float (&yx)[4], const float (&yy)[4], int cnty,
                                                   float &best, int &edge) const {
        best = 0.0f; edge = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (i < cntx) {
                float nx = sm[SC::WNX + 4 * x + i], ny = sm[SC::WNY + 4 * x + i];
                float lo = dot2(nx, ny, yx[0], yy[0]);
#pragma unroll
                for (int j = 1; j < 4; ++j)
                    if (j < cnty) lo = fmin_cmp(lo, dot2(nx, ny, yx[j], yy[j]));
                float sep = lo - sm[SC::WOFF + 4 * x + i];
                if (i == 0 || sep > best) { best = sep; edge = i; }
            }
        }
    }

    __device__ unsigned manifold_pp(int a, int b, Manifold (&m)[2]) const {
        const int cnta = flag_nverts(smu[SC::BFL + a]), cntb = flag_nverts(smu[SC::BFL + b]);
        float ax[4], ay[4], bx[4], by[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            ax[k] = sm[SC::WVX + 4 * a + k]; ay[k] = sm[SC::WVY + 4 * a + k];
            bx[k] = sm[SC::WVX + 4 * b + k]; by[k] = sm[SC::WVY + 4 * b + k];
        }
        float sa, sb; int ea, eb;
        max_separation(a, cnta, bx, by, cntb, sa, ea);
        max_separation(b, cntb, ax, ay, cnta, sb, eb);
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
        const float cx = sm[SC::BX + b], cy = sm[SC::BY + b], r = sm[SC::RAD + (b - SC::P)];
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
        const float ax = sm[SC::BX + a], ay = sm[SC::BY + a], ra = sm[SC::RAD + (a - SC::P)];
        const float dx = sm[SC::BX + b] - ax, dy = sm[SC::BY + b] - ay, rb = sm[SC::RAD + (b - SC::P)];
        const float dist = sqrtf(dot2(dx, dy, dx, dy));
        if (dist < 1e-9f) { m.nx = 0.0f; m.ny = 1.0f; }
        else { const float inv = 1.0f / dist; m.nx = dx * inv; m.ny = dy * inv; }
        m.pen = (ra + rb) - dist;
        m.px = __fmaf_rn(ra, m.nx, ax); m.py = __fmaf_rn(ra, m.ny, ay);
        return m.pen > 0.0f ? 1u : 0u;
    }

    // ---- contact pre-step for one manifold of pair (a, b): writes the manifold part of record k
    __device__ __forceinline__ void prestep_manifold(int k, int mi, int a, int b, const Manifold &m, float acc_n, float acc_t, float er) {
        const float rax = m.px - sm[SC::BX + a], ray = m.py - sm[SC::BY + a];
        const float rbx = m.px - sm[SC::BX + b], rby = m.py - sm[SC::BY + b];
        const float ma = sm[SC::BIM + a], mb = sm[SC::BIM + b], ia = sm[SC::BII + a], ib = sm[SC::BII + b];
        const float tx = -m.ny, ty = m.nx;
        const float rna = cross2(rax, ray, m.nx, m.ny), rnb = cross2(rbx, rby, m.nx, m.ny);
        const float rta = cross2(rax, ray, tx, ty), rtb = cross2(rbx, rby, tx, ty);
        float kn = ma + mb; kn = __fmaf_rn(ia * rna, rna, kn); kn = __fmaf_rn(ib * rnb, rnb, kn);
        float kt = ma + mb; kt = __fmaf_rn(ia * rta, rta, kt); kt = __fmaf_rn(ib * rtb, rtb, kt);
        // normal approach speed before warm starting
        float vn0 = dot2(m.nx, m.ny, sm[SC::BVX + b] - sm[SC::BVX + a], sm[SC::BVY + b] - sm[SC::BVY + a]);
        vn0 = __fmaf_rn(sm[SC::BW + b], rnb, vn0);
        vn0 = __fmaf_rn(-sm[SC::BW + a], rna, vn0);
        const float depth = fmax_cmp(m.pen - prm.slop, 0.0f);
        const float bounce = (vn0 < -prm.rest_thr) ? (-er * vn0) : 0.0f;
        const int f = R_M0 + mi * M_WORDS;
        rec_st(f + M_RNA, k, rna); rec_st(f + M_RNB, k, rnb); rec_st(f + M_RTA, k, rta); rec_st(f + M_RTB, k, rtb);
        rec_st(f + M_MASSN, k, 1.0f / kn); rec_st(f + M_MASST, k, 1.0f / kt);
        rec_st(f + M_TARGET, k, bounce + prm.contact_alpha * depth);
        rec_st(f + M_CORR, k, (prm.contact_beta * depth) / (ma + mb));
        rec_st(f + M_ACCN, k, acc_n); rec_st(f + M_ACCT, k, acc_t);
    }

    // ---- one visit of contact pair record k.  MODE 0: warm start, 1: solver iteration, 2: positional correction
    template <int MODE>
    __device__ __forceinline__ void visit_pair(int k, uint32_t ab) {
        const int a = ab & 31, b = (ab >> 5) & 31;
        const unsigned amask = (ab >> 10) & 3u;
        const bool dyn_a = (ab >> 26) & 1u, dyn_b = (ab >> 27) & 1u;
        const float nx = rec_ld(R_NX, k), ny = rec_ld(R_NY, k);
        const float ma = sm[SC::BIM + a], mb = sm[SC::BIM + b];
        if (MODE == 2) {
            float xa = sm[SC::BX + a], ya = sm[SC::BY + a], xb = sm[SC::BX + b], yb = sm[SC::BY + b];
#pragma unroll
            for (int mi = 0; mi < 2; ++mi) {
                if (amask & (1u << mi)) {
                    const float corr = rec_ld(R_M0 + mi * M_WORDS + M_CORR, k);
                    const float ca = ma * corr, cb = mb * corr;
                    xa = __fmaf_rn(-ca, nx, xa); ya = __fmaf_rn(-ca, ny, ya);
                    xb = __fmaf_rn(cb, nx, xb); yb = __fmaf_rn(cb, ny, yb);
                }
            }
            if (dyn_a) { sm[SC::BX + a] = xa; sm[SC::BY + a] = ya; }
            if (dyn_b) { sm[SC::BX + b] = xb; sm[SC::BY + b] = yb; }
            return;
        }
        const float ia = sm[SC::BII + a], ib = sm[SC::BII + b];
        const float tx = -ny, ty = nx;
        const float mu = rec_ld(R_MU, k);
        float vax = sm[SC::BVX + a], vay = sm[SC::BVY + a], wa = sm[SC::BW + a];
        float vbx = sm[SC::BVX + b], vby = sm[SC::BVY + b], wb = sm[SC::BW + b];
#pragma unroll
        for (int mi = 0; mi < 2; ++mi) {
            if (amask & (1u << mi)) {
                const int f = R_M0 + mi * M_WORDS;
                const float rna = rec_ld(f + M_RNA, k), rnb = rec_ld(f + M_RNB, k);
                const float rta = rec_ld(f + M_RTA, k), rtb = rec_ld(f + M_RTB, k);
                const float wna = ia * rna, wnb = ib * rnb, wta = ia * rta, wtb = ib * rtb;
                float accn = rec_ld(f + M_ACCN, k), acct = rec_ld(f + M_ACCT, k);
                float dn, dt_;
                if (MODE == 0) { dn = accn; }
                else {
                    float vn = dot2(nx, ny, vbx - vax, vby - vay);
                    vn = __fmaf_rn(wb, rnb, vn);
                    vn = __fmaf_rn(-wa, rna, vn);
                    const float lam = (rec_ld(f + M_TARGET, k) - vn) * rec_ld(f + M_MASSN, k);
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
                    const float lam = (-vt) * rec_ld(f + M_MASST, k);
                    const float lim = mu * accn;
                    const float nw = fmax_cmp(fmin_cmp(acct + lam, lim), -lim);
                    dt_ = nw - acct; acct = nw;
                }
                {
                    const float px = dt_ * tx, py = dt_ * ty;
                    vax = __fmaf_rn(-ma, px, vax); vay = __fmaf_rn(-ma, py, vay); wa = __fmaf_rn(-wta, dt_, wa);
                    vbx = __fmaf_rn(mb, px, vbx); vby = __fmaf_rn(mb, py, vby); wb = __fmaf_rn(wtb, dt_, wb);
                }
                if (MODE == 1) { rec_st(f + M_ACCN, k, accn); rec_st(f + M_ACCT, k, acct); }
            }
        }
        if (dyn_a) { sm[SC::BVX + a] = vax; sm[SC::BVY + a] = vay; sm[SC::BW + a] = wa; }
        if (dyn_b) { sm[SC::BVX + b] = vbx; sm[SC::BVY + b] = vby; sm[SC::BW + b] = wb; }
    }

    template <int MODE>
    __device__ __forceinline__ void sweep_pairs(int nrec, int max_level, uint32_t my_ab) {
        for (int lvl = 1; lvl <= max_level; ++lvl) {
            if (lane < nrec && ((my_ab >> 19) & 127u) == (unsigned)lvl) visit_pair<MODE>(lane, my_ab);
            if (nrec > G) {
                for (int k = lane + G; k < nrec; k += G) {
                    const uint32_t ab = __float_as_uint(rec_ld(R_AB, k));
                    if (((ab >> 19) & 127u) == (unsigned)lvl) visit_pair<MODE>(k, ab);
                }
            }
            g.sync();
        }
    }

    // ---- joints.  MODE 0: warm start, 1: solver iteration, 2: positional correction, 3: motor
    template <int MODE>
    __device__ __forceinline__ void visit_joint(int j, uint32_t jab, const uint32_t *lv) {
        const int a = jab & 255, b = (jab >> 8) & 255;
        const bool dyn_a = smu[SC::BFL + a] & F_DYNAMIC, dyn_b = smu[SC::BFL + b] & F_DYNAMIC;
        float *jn = sm + SC::JNT;
        if (MODE == 3) {
            const float A = fmax_cmp(fmin_cmp(sm[SC::ACT + ((jab >> 16) & 255)], 1.0f), -1.0f);
            const float speed = __uint_as_float(lv[SC::LV_JOINT + 8 * j + 5]), power = __uint_as_float(lv[SC::LV_JOINT + 8 * j + 6]);
            const float wa = sm[SC::BW + a], wb = sm[SC::BW + b];
            const float arg = __fmaf_rn(-speed, A, wa - wb) * prm.motor_rho;
            const float jr = power * tanh_spec(arg);
            if (dyn_a) sm[SC::BW + a] = __fmaf_rn(-jr, sm[SC::BII + a], wa);
            if (dyn_b) sm[SC::BW + b] = __fmaf_rn(jr, sm[SC::BII + b], wb);
            return;
        }
        const float ma = sm[SC::BIM + a], mb = sm[SC::BIM + b];
        if (MODE == 2) {
            const float cx = jn[JA_CX * SC::J + j], cy = jn[JA_CY * SC::J + j];
            if (dyn_a) { sm[SC::BX + a] = __fmaf_rn(ma, cx, sm[SC::BX + a]); sm[SC::BY + a] = __fmaf_rn(ma, cy, sm[SC::BY + a]); }
            if (dyn_b) { sm[SC::BX + b] = __fmaf_rn(-mb, cx, sm[SC::BX + b]); sm[SC::BY + b] = __fmaf_rn(-mb, cy, sm[SC::BY + b]); }
            return;
        }
        const float ia = sm[SC::BII + a], ib = sm[SC::BII + b];
        const float rax = jn[JA_RAX * SC::J + j], ray = jn[JA_RAY * SC::J + j];
        const float rbx = jn[JA_RBX * SC::J + j], rby = jn[JA_RBY * SC::J + j];
        float vax = sm[SC::BVX + a], vay = sm[SC::BVY + a], wa = sm[SC::BW + a];
        float vbx = sm[SC::BVX + b], vby = sm[SC::BVY + b], wb = sm[SC::BW + b];
        float lx, ly;
        if (MODE == 0) { lx = jn[JA_ACCX * SC::J + j]; ly = jn[JA_ACCY * SC::J + j]; }
        else {
            const float cx = __fmaf_rn(-wb, rby, vbx) - __fmaf_rn(-wa, ray, vax);
            const float cy = __fmaf_rn(wb, rbx, vby) - __fmaf_rn(wa, rax, vay);
            const float rx = -(cx + jn[JA_BX * SC::J + j]), ry = -(cy + jn[JA_BY * SC::J + j]);
            const float i11 = jn[JA_I11 * SC::J + j], i12 = jn[JA_I12 * SC::J + j], i22 = jn[JA_I22 * SC::J + j];
            lx = __fmaf_rn(i11, rx, i12 * ry);
            ly = __fmaf_rn(i12, rx, i22 * ry);
            jn[JA_ACCX * SC::J + j] = jn[JA_ACCX * SC::J + j] + lx;
            jn[JA_ACCY * SC::J + j] = jn[JA_ACCY * SC::J + j] + ly;
        }
        if (dyn_a) {
            sm[SC::BVX + a] = __fmaf_rn(-ma, lx, vax); sm[SC::BVY + a] = __fmaf_rn(-ma, ly, vay);
            sm[SC::BW + a] = __fmaf_rn(-ia, cross2(rax, ray, lx, ly), wa);
        }
        if (dyn_b) {
            sm[SC::BVX + b] = __fmaf_rn(mb, lx, vbx); sm[SC::BVY + b] = __fmaf_rn(mb, ly, vby);
            sm[SC::BW + b] = __fmaf_rn(ib, cross2(rbx, rby, lx, ly), wb);
        }
    }

    template <int MODE>
    __device__ __forceinline__ void sweep_joints(int max_level, uint32_t my_jab, const uint32_t *lv) {
        if (SC::J == 0) return;
        for (int lvl = 1; lvl <= max_level; ++lvl) {
            for (int j = lane, r = 0; j < SC::J; j += G, ++r) {
                const uint32_t jab = (r == 0) ? my_jab : smu[SC::JNT + JA_AB * SC::J + j];
                if (((jab >> 24) & 1u) && ((jab >> 25) & 7u) == (unsigned)lvl) visit_joint<MODE>(j, jab, lv);
            }
            g.sync();
        }
    }

    // ---- one environment step.  Returns through meta[]: step_count, episode_count, level_id, status, nwarm
    __device__ void step(int e, int s, int (&meta)[5], unsigned (&cnt)[8]) {
        const uint32_t *lv = prm.levels + (size_t)meta[2] * SC::LV_WORDS;
        // frozen env: reports done, nothing else
        if (meta[3] & 1) {
            if (lane == 0) { prm.reward[(size_t)s * prm.n_envs + e] = 0.0f; prm.done[(size_t)s * prm.n_envs + e] = 1; }
            return;
        }
        // actions of this step
        for (int i = lane; i < prm.n_actions; i += G) sm[SC::ACT + i] = prm.actions[((size_t)s * prm.n_envs + e) * prm.n_actions + i];
        // gravity, rotation, circle boxes
        for (int i = lane; i < SC::N; i += G) {
            const uint32_t fl = smu[SC::BFL + i];
            if ((fl & F_ACTIVE) && (fl & F_DYNAMIC)) sm[SC::BVY + i] = sm[SC::BVY + i] + prm.gdt;
            float c, sn;
            sincos_spec(sm[SC::BTH + i], c, sn);
            sm[SC::BC + i] = c; sm[SC::BS + i] = sn;
            if (i >= SC::P) {
                const float r = sm[SC::RAD + (i - SC::P)], x = sm[SC::BX + i], y = sm[SC::BY + i];
                sm[SC::AMINX + i] = x - r; sm[SC::AMINY + i] = y - r; sm[SC::AMAXX + i] = x + r; sm[SC::AMAXY + i] = y + r;
            }
        }
        g.sync();
        // world-frame polygon vertices, normals, face offsets
        for (int v = lane; v < SC::P4; v += G) {
            const int i = v >> 2, k = v & 3;
            if (k < (int)flag_nverts(smu[SC::BFL + i])) {
                const float c = sm[SC::BC + i], sn = sm[SC::BS + i];
                float rx, ry, nx, ny;
                rot2(c, sn, __uint_as_float(lv[SC::LV_PVX + v]), __uint_as_float(lv[SC::LV_PVY + v]), rx, ry);
                rot2(c, sn, __uint_as_float(lv[SC::LV_PNX + v]), __uint_as_float(lv[SC::LV_PNY + v]), nx, ny);
                const float wx = rx + sm[SC::BX + i], wy = ry + sm[SC::BY + i];
                sm[SC::WVX + v] = wx; sm[SC::WVY + v] = wy; sm[SC::WNX + v] = nx; sm[SC::WNY + v] = ny;
                sm[SC::WOFF + v] = dot2(nx, ny, wx, wy);
            }
        }
        // joints: read the packed word once per step
        uint32_t my_jab = 0u;
        if (SC::J > 0 && lane < SC::J) my_jab = lv[SC::LV_JOINT + 8 * lane];
        int jmax = 0;
        if (SC::J > 0) {
            int jl = 0;
            for (int j = lane, r = 0; j < SC::J; j += G, ++r) {
                const uint32_t jab = (r == 0) ? my_jab : lv[SC::LV_JOINT + 8 * j];
                smu[SC::JNT + JA_AB * SC::J + j] = jab;
                if ((jab >> 24) & 1u) jl = max(jl, (int)((jab >> 25) & 7u));
            }
            jmax = g.max_int(jl);
        }
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
            sm[SC::AMINX + i] = x0; sm[SC::AMINY + i] = y0; sm[SC::AMAXX + i] = x1; sm[SC::AMAXY + i] = y1;
        }
        // motors (joint order), thrusters (thruster order)
        sweep_joints<3>(jmax, my_jab, lv);
        if (SC::T > 0) {
            int tl = 0; uint32_t tp = 0u;
            if (lane < SC::T) { tp = lv[SC::LV_THR + 8 * lane]; if ((tp >> 16) & 1u) tl = (tp >> 17) & 7u; }
            const int tmax = g.max_int(tl);
            for (int lvl = 1; lvl <= tmax; ++lvl) {
                if (lane < SC::T && tl == lvl) {
                    const int i = tp & 255;
                    const uint32_t *th = lv + SC::LV_THR + 8 * lane;
                    const float A = fmax_cmp(fmin_cmp(sm[SC::ACT + ((tp >> 8) & 255)], 1.0f), 0.0f);
                    const float c = sm[SC::BC + i], sn = sm[SC::BS + i];
                    float dx, dy, rx, ry;
                    rot2(c, sn, __uint_as_float(th[3]), __uint_as_float(th[4]), dx, dy);
                    rot2(c, sn, __uint_as_float(th[1]), __uint_as_float(th[2]), rx, ry);
                    const float imp = (__uint_as_float(th[5]) * A) * prm.dt;
                    const float jx = imp * dx, jy = imp * dy;
                    const float im = sm[SC::BIM + i];
                    sm[SC::BVX + i] = __fmaf_rn(jx, im, sm[SC::BVX + i]);
                    sm[SC::BVY + i] = __fmaf_rn(jy, im, sm[SC::BVY + i]);
                    sm[SC::BW + i] = __fmaf_rn(cross2(rx, ry, jx, jy), sm[SC::BII + i], sm[SC::BW + i]);
                }
                g.sync();
            }
        }
        // joint pre-step
        for (int j = lane, r = 0; j < SC::J; j += G, ++r) {
            const uint32_t jab = (r == 0) ? my_jab : smu[SC::JNT + JA_AB * SC::J + j];
            float *jn = sm + SC::JNT;
            if (!((jab >> 24) & 1u)) { jn[JA_ACCX * SC::J + j] = 0.0f; jn[JA_ACCY * SC::J + j] = 0.0f; continue; }
            if (!prm.warm_start) { jn[JA_ACCX * SC::J + j] = 0.0f; jn[JA_ACCY * SC::J + j] = 0.0f; }
            const int a = jab & 255, b = (jab >> 8) & 255;
            const uint32_t *jl = lv + SC::LV_JOINT + 8 * j;
            float rax, ray, rbx, rby;
            rot2(sm[SC::BC + a], sm[SC::BS + a], __uint_as_float(jl[1]), __uint_as_float(jl[2]), rax, ray);
            rot2(sm[SC::BC + b], sm[SC::BS + b], __uint_as_float(jl[3]), __uint_as_float(jl[4]), rbx, rby);
            const float ma = sm[SC::BIM + a], mb = sm[SC::BIM + b], ia = sm[SC::BII + a], ib = sm[SC::BII + b];
            const float gx = (sm[SC::BX + b] + rbx) - (sm[SC::BX + a] + rax), gy = (sm[SC::BY + b] + rby) - (sm[SC::BY + a] + ray);
            const float msum = ma + mb;
            float k11 = msum; k11 = __fmaf_rn(ia * ray, ray, k11); k11 = __fmaf_rn(ib * rby, rby, k11);
            float k22 = msum; k22 = __fmaf_rn(ia * rax, rax, k22); k22 = __fmaf_rn(ib * rbx, rbx, k22);
            float k12 = -((ia * rax) * ray); k12 = __fmaf_rn(-(ib * rbx), rby, k12);
            const float det = __fmaf_rn(k11, k22, -(k12 * k12));
            const float inv_det = 1.0f / det;
            jn[JA_RAX * SC::J + j] = rax; jn[JA_RAY * SC::J + j] = ray; jn[JA_RBX * SC::J + j] = rbx; jn[JA_RBY * SC::J + j] = rby;
            jn[JA_I11 * SC::J + j] = k22 * inv_det; jn[JA_I22 * SC::J + j] = k11 * inv_det; jn[JA_I12 * SC::J + j] = -(k12 * inv_det);
            jn[JA_BX * SC::J + j] = prm.joint_alpha * gx; jn[JA_BY * SC::J + j] = prm.joint_alpha * gy;
            const float share = prm.joint_beta / msum;
            jn[JA_CX * SC::J + j] = share * gx; jn[JA_CY * SC::J + j] = share * gy;
        }
        g.sync();

        // bounding-box test over all pairs -> compact list of surviving pairs, in pair order
        int nsurv = 0, ns_pp = 0, ns_pc = 0;
        for (int base = 0; base < SC::NPAIRS; base += G) {
            const int p = base + lane;
            bool keep = false;
            if (p < SC::NPAIRS && ((smu[SC::MASK + (p >> 5)] >> (p & 31)) & 1u)) {
                const int a = ptab[p] & 255, b = ptab[p] >> 8;
                const float mg = prm.aabb_margin;
                keep = !(sm[SC::AMAXX + a] + mg < sm[SC::AMINX + b] || sm[SC::AMAXX + b] + mg < sm[SC::AMINX + a] ||
                         sm[SC::AMAXY + a] + mg < sm[SC::AMINY + b] || sm[SC::AMAXY + b] + mg < sm[SC::AMINY + a]);
            }
            const unsigned bal = g.ballot(keep);
            if (keep) surv()[nsurv + __popc(bal & g.lanes_below())] = (uint8_t)p;
            nsurv += __popc(bal);
            // segment boundaries: survivors below NPP are polygon-polygon, below NPP+NPC polygon-circle
            if (base + G <= SC::NPP) ns_pp = nsurv;
            else if (base < SC::NPP) ns_pp += __popc(bal & ((SC::NPP - base >= 32) ? 0xffffffffu : ((1u << (SC::NPP - base)) - 1u)));
            if (base + G <= SC::NPP + SC::NPC) ns_pc = nsurv;
            else if (base < SC::NPP + SC::NPC) {
                const int lim = SC::NPP + SC::NPC - base;
                ns_pc += __popc(bal & ((lim >= 32) ? 0xffffffffu : ((1u << lim) - 1u)));
            }
        }
        g.sync();
        if (lane == 0) { cnt[4] += ns_pp; cnt[5] += ns_pc - ns_pp; cnt[6] += nsurv - ns_pc; }

        // narrowphase + contact pre-step: survivors of one kind at a time, records in pair order
        int nrec = 0;
        bool t_gb = false, t_gr = false;
        float *trace = prm.trace ? prm.trace + (size_t)e * SC::NSLOTS * 6 : nullptr;
        if (trace) for (int i = lane; i < SC::NSLOTS * 6; i += G) trace[i] = ((i % 6) == 3) ? 1.0f : ((i % 6) == 4 ? -1.0f : 0.0f);
        if (trace) g.sync();
        for (int kind = 0; kind < 3; ++kind) {
            const int lo = kind == 0 ? 0 : (kind == 1 ? ns_pp : ns_pc);
            const int hi = kind == 0 ? ns_pp : (kind == 1 ? ns_pc : nsurv);
            for (int base = lo; base < hi; base += G) {
                const int idx = base + lane;
                unsigned act = 0u;
                Manifold m[2];
                int p = 0, a = 0, b = 0;
                if (idx < hi) {
                    p = surv()[idx]; a = ptab[p] & 255; b = ptab[p] >> 8;
                    if (kind == 0) act = manifold_pp(a, b, m);
                    else if (kind == 1) act = manifold_pc(a, b, m[0]);
                    else act = manifold_cc(a, b, m[0]);
                    // a polygon pair rejected before its manifolds exist leaves its slots at the default
                    if (trace && !(kind == 0 && act == 0u)) {
                        const int slot = (p < SC::NPP) ? 2 * p : SC::NPP + p;
                        const int nm = (kind == 0) ? 2 : 1;
                        for (int mi = 0; mi < nm; ++mi) {
                            float *t = trace + (slot + mi) * 6;
                            t[0] = m[mi].px; t[1] = m[mi].py; t[2] = m[mi].nx; t[3] = m[mi].ny; t[4] = m[mi].pen;
                            t[5] = ((act >> mi) & 1u) ? 1.0f : 0.0f;
                        }
                    }
                }
                const unsigned bal = g.ballot(act != 0u);
                if (act) {
                    const int k = nrec + __popc(bal & g.lanes_below());
                    const uint32_t fa = smu[SC::BFL + a], fb = smu[SC::BFL + b];
                    const uint32_t ra = flag_role(fa), rb = flag_role(fb);
                    t_gb |= (ra == 1u && rb == 2u) || (ra == 2u && rb == 1u);
                    t_gr |= (ra == 1u && rb == 3u) || (ra == 3u && rb == 1u);
                    // accumulated impulses of the previous step, kept per slot while the slot stays active
                    float wacc[4] = { 0.0f, 0.0f, 0.0f, 0.0f };
                    const int wi = widx()[p];
                    if (prm.warm_start && wi != 255) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) wacc[q] = __uint_as_float(warm_ld(1 + q, wi));
                    }
                    const float fra = sm[SC::BFR + a], frb = sm[SC::BFR + b];
                    const float er = fmin_cmp(sm[SC::BRE + a], sm[SC::BRE + b]);
                    const uint32_t ab = (uint32_t)a | ((uint32_t)b << 5) | (act << 10) | ((uint32_t)p << 12) |
                                        (((fa & F_DYNAMIC) ? 1u : 0u) << 26) | (((fb & F_DYNAMIC) ? 1u : 0u) << 27);
                    rec_st(R_AB, k, __uint_as_float(ab));
                    rec_st(R_NX, k, (act & 1u) ? m[0].nx : m[1].nx);
                    rec_st(R_NY, k, (act & 1u) ? m[0].ny : m[1].ny);
                    rec_st(R_MU, k, sqrtf(__fmaf_rn(fra, fra, frb * frb)));
                    if (act & 1u) prestep_manifold(k, 0, a, b, m[0], wacc[0], wacc[1], er);
                    if (act & 2u) prestep_manifold(k, 1, a, b, m[1], wacc[2], wacc[3], er);
                }
                nrec += __popc(bal);
            }
        }
        const bool touch_gb = g.any(t_gb), touch_gr = g.any(t_gr);
        g.sync();

        // levels of the contact pair records (canonical order = record order)
        uint32_t my_ab = 0u;
        int max_level = 0;
        if (nrec <= G) {
            int lvl = 0;
            if (lane < nrec) { my_ab = __float_as_uint(rec_ld(R_AB, lane)); lvl = 1; }
            const int a = my_ab & 31, b = (my_ab >> 5) & 31;
            const bool da = (my_ab >> 26) & 1u, db = (my_ab >> 27) & 1u;
            for (int q = 0; q < nrec; ++q) {
                const uint32_t abq = g.shflu(my_ab, q);
                const int lq = g.shfl(lvl, q);
                const int aq = abq & 31, bq = (abq >> 5) & 31;
                const bool hit = (da && (a == aq || a == bq)) || (db && (b == aq || b == bq));
                if (q < lane && lane < nrec && hit) lvl = max(lvl, lq + 1);
            }
            my_ab |= (uint32_t)lvl << 19;
            if (lane < nrec) rec_st(R_AB, lane, __uint_as_float(my_ab));
            max_level = g.max_int(lvl);
        } else {
            // rare: more active pairs than lanes; one lane assigns levels with a per-body table
            if (lane == 0) {
                uint8_t *bl = surv();   // the survivor list is no longer needed
                for (int i = 0; i < SC::N; ++i) bl[i] = 0;
                for (int k = 0; k < nrec; ++k) {
                    uint32_t ab = __float_as_uint(rec_ld(R_AB, k));
                    const int a = ab & 31, b = (ab >> 5) & 31;
                    int lvl = 1;
                    if ((ab >> 26) & 1u) lvl = max(lvl, bl[a] + 1);
                    if ((ab >> 27) & 1u) lvl = max(lvl, bl[b] + 1);
                    if ((ab >> 26) & 1u) bl[a] = (uint8_t)lvl;
                    if ((ab >> 27) & 1u) bl[b] = (uint8_t)lvl;
                    rec_st(R_AB, k, __uint_as_float(ab | ((uint32_t)lvl << 19)));
                    max_level = max(max_level, lvl);
                }
            }
            __threadfence_block();
            g.sync();
            max_level = g.shfl(max_level, 0);
            if (lane < nrec) my_ab = __float_as_uint(rec_ld(R_AB, lane));
        }
        g.sync();

        // warm start: contacts, then joints
        sweep_pairs<0>(nrec, max_level, my_ab);
        if (SC::J > 0) sweep_joints<0>(jmax, my_jab, lv);
        // solver iterations: joints, then contacts
        for (int it = 0; it < prm.solver_iters; ++it) {
            sweep_joints<1>(jmax, my_jab, lv);
            sweep_pairs<1>(nrec, max_level, my_ab);
        }
        // Euler step with the solved velocities
        bool finite = true;
        for (int i = lane; i < SC::N; i += G) {
            if (smu[SC::BFL + i] & F_ACTIVE) {
                sm[SC::BX + i] = __fmaf_rn(prm.dt, sm[SC::BVX + i], sm[SC::BX + i]);
                sm[SC::BY + i] = __fmaf_rn(prm.dt, sm[SC::BVY + i], sm[SC::BY + i]);
                sm[SC::BTH + i] = __fmaf_rn(prm.dt, sm[SC::BW + i], sm[SC::BTH + i]);
            }
        }
        g.sync();
        sweep_pairs<2>(nrec, max_level, my_ab);
        sweep_joints<2>(jmax, my_jab, lv);
        for (int i = lane; i < SC::N; i += G)
            finite = finite && finite_bits(sm[SC::BX + i]) && finite_bits(sm[SC::BY + i]) && finite_bits(sm[SC::BTH + i]) &&
                     finite_bits(sm[SC::BVX + i]) && finite_bits(sm[SC::BVY + i]) && finite_bits(sm[SC::BW + i]);
        finite = !g.any(!finite);

        // accumulated impulses of this step become the warm list of the next one
        for (int i = lane; i < (SC::NPAIRS + 3) / 4; i += G) smu[SC::WIDX + i] = 0xffffffffu;
        g.sync();
        int nman = 0;
        for (int k = lane; k < nrec; k += G) {
            const uint32_t ab = (k == lane) ? my_ab : __float_as_uint(rec_ld(R_AB, k));
            const int p = (ab >> 12) & 127;
            const unsigned am = (ab >> 10) & 3u;
            warm_st(0, k, (uint32_t)p);
            warm_st(1, k, (am & 1u) ? __float_as_uint(rec_ld(R_M0 + M_ACCN, k)) : 0u);
            warm_st(2, k, (am & 1u) ? __float_as_uint(rec_ld(R_M0 + M_ACCT, k)) : 0u);
            warm_st(3, k, (am & 2u) ? __float_as_uint(rec_ld(R_M0 + M_WORDS + M_ACCN, k)) : 0u);
            warm_st(4, k, (am & 2u) ? __float_as_uint(rec_ld(R_M0 + M_WORDS + M_ACCT, k)) : 0u);
            widx()[p] = (uint8_t)k;
            nman += __popc(am);
        }
        meta[4] = nrec;
        if (lane == 0) cnt[7] += nrec;

        // reward, termination, counters, auto-reset
        meta[0] += 1;
        const bool timeout = prm.max_episode_steps > 0 && meta[0] >= prm.max_episode_steps;
        float reward = (float)((int)touch_gb - (int)touch_gr);
        bool done = touch_gb || touch_gr || timeout;
        if (!finite) { reward = 0.0f; done = true; meta[3] |= 1; if (lane == 0) cnt[0] += 1; }
        if (lane == 0) {
            prm.reward[(size_t)s * prm.n_envs + e] = reward;
            prm.done[(size_t)s * prm.n_envs + e] = done ? 1 : 0;
            cnt[3] += 1;
        }
        cnt[2] += nman;
        g.sync();
        if (done && prm.auto_reset != 0) {
            meta[1] += 1;
            if (prm.auto_reset == 2) {
                const unsigned long long h = mix64(prm.seed + ((unsigned long long)(prm.env_offset + e) + 1ULL) * 0x9E3779B97F4A7C15ULL +
                                                   (unsigned long long)meta[1] * 0xD1B54A32D192ED03ULL);
                const int nl = (int)(h % (unsigned long long)prm.n_levels);
                if (nl != meta[2]) { meta[2] = nl; load_level_consts(prm.levels + (size_t)nl * SC::LV_WORDS); }
            }
            load_level_pose(prm.levels + (size_t)meta[2] * SC::LV_WORDS);
            meta[0] = 0; meta[3] = 0; meta[4] = 0;
            if (lane == 0) cnt[1] += 1;
            g.sync();
        }
    }

    // ---- whole launch for one scene
    __device__ void run(int e) {
        uint32_t *st = prm.state + (size_t)e * SC::ST_WORDS;
        int meta[5];
#pragma unroll
        for (int i = 0; i < 5; ++i) meta[i] = (int)st[SC::ST_META + i];
        for (int i = lane; i < 6 * SC::N; i += G) smu[SC::BX + i] = st[SC::ST_BODY + i];
        for (int i = lane; i < SC::J; i += G) {
            smu[SC::JNT + JA_ACCX * SC::J + i] = st[SC::ST_JACC + 2 * i];
            smu[SC::JNT + JA_ACCY * SC::J + i] = st[SC::ST_JACC + 2 * i + 1];
        }
        for (int i = lane; i < (SC::NPAIRS + 3) / 4; i += G) smu[SC::WIDX + i] = 0xffffffffu;
        load_level_consts(prm.levels + (size_t)meta[2] * SC::LV_WORDS);
        g.sync();
        for (int k = lane; k < meta[4]; k += G) {
            const uint32_t p = st[SC::ST_WARM + kWarmWords * k];
            warm_st(0, k, p);
#pragma unroll
            for (int q = 1; q < 5; ++q) warm_st(q, k, st[SC::ST_WARM + kWarmWords * k + q]);
            widx()[p] = (uint8_t)k;
        }
        g.sync();
        unsigned cnt[8] = { 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u };
        for (int s = 0; s < prm.n_steps; ++s) { step(e, s, meta, cnt); g.sync(); }
        // write back
        for (int i = lane; i < 6 * SC::N; i += G) st[SC::ST_BODY + i] = smu[SC::BX + i];
        for (int i = lane; i < SC::J; i += G) {
            st[SC::ST_JACC + 2 * i] = smu[SC::JNT + JA_ACCX * SC::J + i];
            st[SC::ST_JACC + 2 * i + 1] = smu[SC::JNT + JA_ACCY * SC::J + i];
        }
        if (lane < 5) st[SC::ST_META + lane] = (uint32_t)meta[lane];
        for (int k = lane; k < meta[4]; k += G) {
#pragma unroll
            for (int q = 0; q < 5; ++q) st[SC::ST_WARM + kWarmWords * k + q] = warm_ld(q, k);
        }
        // counters: lane 0 holds the event counts, every lane holds its share of the manifold count
        unsigned nm = cnt[2];
        for (int off = G / 2; off > 0; off >>= 1) nm += __shfl_down_sync(g.mask, nm, off, G);
        if (lane == 0) {
            cnt[2] = nm;
#pragma unroll
            for (int q = 0; q < 8; ++q) if (cnt[q]) atomicAdd(prm.counters + q, (unsigned long long)cnt[q]);
        }
    }
};

template <class SC>
__device__ __forceinline__ uint16_t pair_code(int p) {
    int a, b;
    if (p < SC::NPP) { int i = 0, rem = p; while (rem >= SC::P - 1 - i) { rem -= SC::P - 1 - i; ++i; } a = i; b = i + 1 + rem; }
    else if (p < SC::NPP + SC::NPC) { const int q = p - SC::NPP; a = q / SC::C; b = SC::P + q % SC::C; }
    else { int i = 0, rem = p - SC::NPP - SC::NPC; while (rem >= SC::C - 1 - i) { rem -= SC::C - 1 - i; ++i; } a = SC::P + i; b = SC::P + i + 1 + rem; }
    return (uint16_t)(a | (b << 8));
}

template <class SC, int G>
__global__ void __launch_bounds__(kBlockThreads) k2d_step_kernel(const StepParams prm) {
    extern __shared__ __align__(16) uint32_t smem_raw[];
    constexpr int GPB = kBlockThreads / G;
    uint16_t *ptab = reinterpret_cast<uint16_t *>(smem_raw);
    for (int p = threadIdx.x; p < SC::NPAIRS; p += kBlockThreads) ptab[p] = pair_code<SC>(p);
    __syncthreads();
    const int gib = threadIdx.x / G;
    const int slot = blockIdx.x * GPB + gib, nslots = gridDim.x * GPB;
    uint32_t *region = smem_raw + SC::PTAB_WORDS + gib * region_words<SC, G>();
    uint32_t *scratch = SC::OVF > 0 ? prm.scratch + (size_t)slot * SC::SCRATCH_WORDS : nullptr;
    Scene<SC, G> scene(region, ptab, scratch, prm);
    for (int e = slot; e < prm.n_envs; e += nslots) { scene.run(e); scene.g.sync(); }
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

// ---------------------------------------------------------------- observation kernel: one warp per env
template <class SC>
__global__ void __launch_bounds__(kBlockThreads) k2d_obs_kernel(const uint32_t *state, const uint32_t *levels, float *obs,
                                                                int n_envs, int n_actions, int n_polygons, int n_circles,
                                                                int n_joints, int n_thrusters) {
    __shared__ float cs[kBlockThreads / 32][2 * SC::N];
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int e = blockIdx.x * (kBlockThreads / 32) + w;
    if (e >= n_envs) return;
    const uint32_t *st = state + (size_t)e * SC::ST_WORDS;
    const uint32_t *lv = levels + (size_t)st[SC::ST_META + 2] * SC::LV_WORDS;
    const float *stf = reinterpret_cast<const float *>(st);
    const float *lvf = reinterpret_cast<const float *>(lv);
    for (int i = lane; i < SC::N; i += 32) {
        float c, s;
        sincos_spec(stf[2 * SC::N + i], c, s);
        cs[w][i] = c; cs[w][SC::N + i] = s;
    }
    __syncwarp();
    const int n_shapes = n_polygons + n_circles;
    const int jw = 11 + n_actions;
    const int width = n_shapes * 29 + 2 * n_joints * jw + 6 * n_thrusters;
    float *o = obs + (size_t)e * width;
    for (int idx = lane; idx < width; idx += 32) {
        float v = 0.0f;
        if (idx < n_shapes * 29) {
            const int ci = idx / 29, f = idx - ci * 29;
            const int i = ci < n_polygons ? ci : SC::P + (ci - n_polygons);     // internal shape index
            const uint32_t fl = lv[SC::LV_FLAGS + i];
            if (fl & F_ACTIVE) {
                const int nv = flag_nverts(fl);
                if (f == 0) v = stf[i];
                else if (f == 1) v = stf[SC::N + i];
                else if (f == 2) v = stf[3 * SC::N + i];
                else if (f == 3) v = stf[4 * SC::N + i];
                else if (f == 4) v = lvf[SC::LV_IM + i];
                else if (f == 5) v = lvf[SC::LV_II + i];
                else if (f == 6) v = lvf[SC::LV_DENS + i];
                else if (f == 7) v = tanh_spec(stf[5 * SC::N + i] * 0.1f);
                else if (f < 12) v = (flag_role(fl) == (uint32_t)(f - 8)) ? 1.0f : 0.0f;
                else if (f == 12) v = cs[w][SC::N + i];
                else if (f == 13) v = cs[w][i];
                else if (f == 14) v = lvf[SC::LV_FR + i];
                else if (f == 15) v = lvf[SC::LV_RE + i];
                else if (f == 16) v = i < SC::P ? 1.0f : 0.0f;
                else if (f == 17) v = i < SC::P ? 0.0f : 1.0f;
                else if (f == 18) v = i < SC::P ? 0.0f : lvf[SC::LV_RAD + (i - SC::P)];
                else if (f < 27) {
                    const int q = f - 19, k = q >> 1;
                    if (i < SC::P && k < nv) v = (q & 1) ? lvf[SC::LV_PVY + 4 * i + k] : lvf[SC::LV_PVX + 4 * i + k];
                } else if (i < SC::P) v = ((f == 27) == (nv == 3)) ? 1.0f : 0.0f;
            }
        } else if (idx < n_shapes * 29 + 2 * n_joints * jw) {
            const int q = idx - n_shapes * 29;
            const int row = q / jw, f = q - row * jw;
            const int j = row >> 1, d = row & 1;
            const uint32_t *jl = lv + SC::LV_JOINT + 8 * j;
            const uint32_t jab = jl[0];
            if ((jab >> 28) & 1u) {
                const int a = jab & 255, b = (jab >> 8) & 255;
                const int from = d ? b : a, to = d ? a : b;
                if (f == 0) v = 1.0f;
                else if (f >= 2 && f < 6) { const int side = ((f - 2) >> 1) ^ d; v = __uint_as_float(jl[1 + 2 * side + ((f - 2) & 1)]); }
                else if (f == 6) v = __uint_as_float(jl[6]);
                else if (f == 7) v = __uint_as_float(jl[5]);
                else if (f >= 9 && f < 9 + n_actions) v = ((int)((jab >> 16) & 255) == f - 9) ? 1.0f : 0.0f;
                else if (f == 9 + n_actions) v = __fmaf_rn(cs[w][SC::N + to], cs[w][from], -(cs[w][to] * cs[w][SC::N + from]));
                else if (f == 10 + n_actions) v = __fmaf_rn(cs[w][to], cs[w][from], cs[w][SC::N + to] * cs[w][SC::N + from]);
            }
        } else {
            const int q = idx - n_shapes * 29 - 2 * n_joints * jw;
            const int t = q / 6, f = q - t * 6;
            const uint32_t *th = lv + SC::LV_THR + 8 * t;
            const uint32_t tp = th[0];
            if ((tp >> 20) & 1u) {
                const int i = tp & 255;
                float dx, dy;
                rot2(cs[w][i], cs[w][SC::N + i], __uint_as_float(th[3]), __uint_as_float(th[4]), dx, dy);
                if (f == 0) v = 1.0f;
                else if (f == 1) v = __uint_as_float(th[1]);
                else if (f == 2) v = __uint_as_float(th[2]);
                else if (f == 3) v = __uint_as_float(th[5]);
                else if (f == 4) v = dy;
                else v = dx;
            }
        }
        o[idx] = v;
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
