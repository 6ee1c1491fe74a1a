/*
 * k2d_oracle.c -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, scalar CPU implementation of one environment step of the
 * batched 2D rigid-body engine described in the Kinetix / Jax2D paper
 * (arxiv 2410.23208, Appendix "Jax2D"), written from the paper's text and
 * equations.  Only tests, the smoke check and the benchmark's CPU-baseline
 * leg may load this file; the CUDA library shares no code with it.
 *
 * One scene at a time, no blocking, no reordering: every loop runs in the
 * order the paper's Algorithm 1 gives (gravity, manifolds, motors, thrusters,
 * warm start, solver iterations of joints-then-contacts, Euler step).  Where
 * the paper is silent the reading taken is stated next to the code.
 *
 * Arithmetic: `real` is float (the parity build) or double (build with
 * -DK2D_ORACLE_F64: same statements, used by closed-form pins that need more
 * digits than fp32 gives).  Every +,-,*,/,sqrt is a separately rounded IEEE
 * operation (compile with -ffp-contract=off); a fused multiply-add is used
 * exactly where the code says R_FMA.  min/max are written as comparisons so
 * that NaN and signed-zero behaviour is fixed by the language.
 *
 * Parity pins (see tests/): free fall closed form, two-circle collision
 * momentum/restitution, circle-plane and corner distances by brute force,
 * polygon overlap by Sutherland-Hodgman brute force, resting box impulse
 * m*g*dt, sliding-block Coulomb deceleration, pendulum period and energy,
 * motor recurrence, thruster closed form, fixed-joint common angular velocity
 * and error decay, joint-limit stops, multi-discrete codes, dense reward of a
 * body at constant speed, rendered areas and draw order, solver invariants,
 * splitmix64 vectors, sincos/tanh against libm.  The whole step has no Jax2D trajectory
 * to compare with: "parity unpinned" against the paper's own implementation.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef K2D_ORACLE_F64
typedef double real;
#define R_FMA(a, b, c) fma((a), (b), (c))
#define R_SQRT(a) sqrt(a)
#else
typedef float real;
#define R_FMA(a, b, c) fmaf((a), (b), (c))
#define R_SQRT(a) sqrtf(a)
#endif
#define RC(x) ((real)(x))

#define MAX_VERTS 4
#define ROLE_NONE 0
#define ROLE_GREEN 1
#define ROLE_BLUE 2
#define ROLE_RED 3
#define RESET_NONE 0
#define RESET_SAME 1
#define RESET_POOL 2
#define STATUS_NONFINITE 1

typedef struct { real x, y; } vec2;

/* ---- configuration and raw level description (filled by the caller) ---- */
typedef struct {
    int32_t n_polygons, n_circles, n_joints, n_thrusters, n_actions, n_levels, n_envs;
    int32_t solver_iters, warm_start, auto_reset, max_episode_steps, broadphase, discrete_actions, frame_skip, solver_batch;
    real dt, gravity_y, contact_alpha, contact_beta, slop, restitution_threshold, face_tol;
    real joint_alpha, joint_beta, motor_rho, aabb_margin, joint_gamma, dense_kappa;
    uint64_t seed;
    int64_t env_offset;
} ref_config;

typedef struct {
    const real *poly_verts;      /* [L][P][4][2] body-frame vertices, CCW, centroid at origin */
    const int32_t *poly_nverts;  /* [L][P] 3 or 4 */
    const real *circle_radius;   /* [L][C] */
    const real *pos, *angle, *vel, *angvel;         /* [L][N][2], [L][N], [L][N][2], [L][N] */
    const real *density, *friction, *restitution;   /* [L][N] */
    const int32_t *is_static, *role, *active;       /* [L][N] */
    const int32_t *joint_a, *joint_b;               /* [L][J] */
    const real *joint_anchor_a, *joint_anchor_b;    /* [L][J][2] body-frame */
    const real *motor_speed, *motor_power;          /* [L][J] */
    const int32_t *motor_binding, *joint_active;    /* [L][J] */
    const int32_t *joint_fixed, *joint_limited;     /* [L][J] fixed joint / revolute joint with rotation limits */
    const real *joint_fixed_angle, *joint_min, *joint_max; /* [L][J] relative rotation (angle a - angle b) held / allowed */
    const int32_t *thr_shape;                       /* [L][T] */
    const real *thr_pos, *thr_rot, *thr_power;      /* [L][T][2], [L][T], [L][T] */
    const int32_t *thr_binding, *thr_active;        /* [L][T] */
} ref_levels;

/* ---- the simulator object: copied levels, derived constants, state ---- */
typedef struct {
    ref_config cfg;
    int P, C, N, J, T, n_pairs, n_pp, n_pc, n_cc, n_slots;
    int *pair_a, *pair_b, *pair_slot; /* canonical pair list */
    /* per level (copied + derived) */
    real *lv_verts, *lv_normals, *lv_edge_len; int32_t *lv_nverts;
    real *lv_radius, *lv_pos, *lv_angle, *lv_vel, *lv_angvel;
    real *lv_density, *lv_friction, *lv_restitution, *lv_inv_mass, *lv_inv_inertia;
    int32_t *lv_static, *lv_role, *lv_active;
    int32_t *lv_joint_a, *lv_joint_b, *lv_motor_binding, *lv_joint_active;
    real *lv_anchor_a, *lv_anchor_b, *lv_motor_speed, *lv_motor_power;
    int32_t *lv_joint_fixed, *lv_joint_limited;
    real *lv_fixed_angle, *lv_joint_min, *lv_joint_max;
    int32_t *lv_thr_shape, *lv_thr_binding, *lv_thr_active;
    real *lv_thr_pos, *lv_thr_rot, *lv_thr_dir, *lv_thr_power;
    uint8_t *lv_collide; /* [L][n_pairs] */
    /* per env state */
    real *pos, *angle, *vel, *angvel;  /* [E][N][2] ... */
    real *acc;        /* [E][n_slots][2] accumulated normal, tangent impulse */
    real *jacc;       /* [E][J][3] accumulated joint impulse: point constraint x, y; fixed joint's angular impulse */
    int32_t *step_count, *episode_count, *level_id, *status;
    /* per env trace of the last step's manifolds: [E][n_slots][6] = px,py,nx,ny,pen,active */
    real *manifold;
    int64_t *counters; /* [8]: nonfinite events, resets, active manifolds (sum), env-steps,
                          pairs past the box test: polygon-polygon, polygon-circle, circle-circle, pairs with an active manifold */
} ref_sim;

typedef struct {
    real *pos, *angle, *vel, *angvel, *acc, *jacc;
    int32_t *step_count, *episode_count, *level_id, *status;
    real *manifold;
    real *inv_mass, *inv_inertia;  /* per LEVEL, [L][N] */
    int32_t *pair_a, *pair_b, *pair_slot;
    uint8_t *collide;              /* per LEVEL, [L][n_pairs] */
    int64_t *counters;
    int32_t n_pairs, n_slots;
} ref_views;

/* ---- exact helpers ---- */
static inline real rmin(real a, real b) { return a < b ? a : b; }
static inline real rmax(real a, real b) { return a > b ? a : b; }
static inline real dot2(vec2 a, vec2 b) { return R_FMA(a.x, b.x, a.y * b.y); }
static inline real cross2(vec2 a, vec2 b) { return R_FMA(a.x, b.y, -(a.y * b.x)); }
static inline vec2 rot2(real c, real s, vec2 v) {
    vec2 o = { R_FMA(c, v.x, -(s * v.y)), R_FMA(s, v.x, c * v.y) };
    return o;
}
static inline vec2 sub2(vec2 a, vec2 b) { vec2 o = { a.x - b.x, a.y - b.y }; return o; }
static inline vec2 perp2(vec2 n) { vec2 o = { -n.y, n.x }; return o; }

/* ---- specified transcendental routines (fp32 build) ----
 * sincos: three-constant Cody-Waite reduction to [-pi/4, pi/4] with FMA, then
 * the Taylor polynomials of sin (degree 9) and cos (degree 10) by Horner.
 * tanh: sign(x) * (1 - t) / (1 + t), t = exp(-2 min(|x|, 10)), exp by
 * reduction to [-ln2/2, ln2/2] and the degree-7 Taylor polynomial.
 * The double build calls libm instead. */
void k2d_ref_sincos(real th, real *c_out, real *s_out) {
#ifdef K2D_ORACLE_F64
    *c_out = cos(th); *s_out = sin(th);
#else
    if (!(fabsf(th) <= 1.0e6f)) { *c_out = NAN; *s_out = NAN; return; }
    const float two_over_pi = 0x1.45f306p-1f;
    const float p1 = 0x1.921fb6p+0f;      /* float(pi/2)              */
    const float p2 = -0x1.777a5cp-25f;        /* float(pi/2 - p1)         */
    const float p3 = -0x1.ee59dap-50f;          /* float(pi/2 - p1 - p2)    */
    float k = rintf(th * two_over_pi);
    float r = fmaf(-k, p1, th);
    r = fmaf(-k, p2, r);
    r = fmaf(-k, p3, r);
    int q = ((int)k) & 3;
    float r2 = r * r;
    float ps = fmaf(0x1.71de3ap-19f, r2, -0x1.a01a02p-13f);
    ps = fmaf(ps, r2, 0x1.111112p-7f);
    ps = fmaf(ps, r2, -0x1.555556p-3f);
    float sp = fmaf(ps * r2, r, r);
    float pc = fmaf(-0x1.27e4fcp-22f, r2, 0x1.a01a02p-16f);
    pc = fmaf(pc, r2, -0x1.6c16c2p-10f);
    pc = fmaf(pc, r2, 0x1.555556p-5f);
    pc = fmaf(pc, r2, -0.5f);
    float cp = fmaf(pc, r2, 1.0f);
    float c, s;
    if (q == 0) { c = cp; s = sp; }
    else if (q == 1) { c = -sp; s = cp; }
    else if (q == 2) { c = -cp; s = -sp; }
    else { c = sp; s = -cp; }
    *c_out = c; *s_out = s;
#endif
}

real k2d_ref_tanh(real x) {
#ifdef K2D_ORACLE_F64
    return tanh(x);
#else
    if (x != x) return x;
    float ax = fabsf(x);
    ax = rmin(ax, 10.0f);
    float y = -2.0f * ax;
    const float log2e = 0x1.715476p+0f;
    const float ln2_hi = 0x1.62e4p-1f;          /* 12 leading bits of ln 2 */
    const float ln2_lo = 0x1.7f7d1cp-20f;     /* ln 2 - ln2_hi           */
    float k = rintf(y * log2e);
    float r = fmaf(-k, ln2_hi, y);
    r = fmaf(-k, ln2_lo, r);
    float p = fmaf(0x1.a01a02p-13f, r, 0x1.6c16c2p-10f);
    p = fmaf(p, r, 0x1.111112p-7f);
    p = fmaf(p, r, 0x1.555556p-5f);
    p = fmaf(p, r, 0x1.555556p-3f);
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    int32_t bits = (((int32_t)k) + 127) << 23;
    float scale; memcpy(&scale, &bits, 4);
    float t = p * scale;
    float v = (1.0f - t) / (1.0f + t);
    return x < 0.0f ? -v : v;
#endif
}

/* splitmix64 finaliser (public domain, S. Vigna): the integer hash that picks
 * the next level on auto-reset. */
uint64_t k2d_ref_mix64(uint64_t z) {
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL;
    z ^= z >> 27; z *= 0x94D049BB133111EBULL;
    z ^= z >> 31;
    return z;
}
static uint64_t reset_hash(uint64_t seed, uint64_t env, uint64_t episode) {
    return k2d_ref_mix64(seed + (env + 1) * 0x9E3779B97F4A7C15ULL + episode * 0xD1B54A32D192ED03ULL);
}

static int is_finite_real(real v) { return (v - v) == RC(0); }

/* ---- collision manifolds (paper: "Collision Manifolds" subsections) ----
 * A manifold is position p, unit normal n (pointing from shape a to shape b)
 * and penetration pen; it is active iff pen > 0. */
typedef struct { vec2 p, n; real pen; int active; } manifold;

/* Circle-circle.  n = (pb - pa)/|pb - pa| (or (0,1) when the centres coincide,
 * a case the paper does not mention), pen = ra + rb - |pb - pa|, p = pa + ra n. */
static void manifold_cc(vec2 pa, real ra, vec2 pb, real rb, manifold *m) {
    vec2 d = sub2(pb, pa);
    real dist = R_SQRT(dot2(d, d));
    vec2 n;
    if (dist < RC(1e-9)) { n.x = RC(0); n.y = RC(1); }
    else { real inv = RC(1) / dist; n.x = d.x * inv; n.y = d.y * inv; }
    m->n = n;
    m->pen = (ra + rb) - dist;
    m->p.x = R_FMA(ra, n.x, pa.x);
    m->p.y = R_FMA(ra, n.y, pa.y);
    m->active = m->pen > RC(0);
}

/* world-frame polygon: vertices w, outward unit edge normals nrm (edge k runs
 * from w[k] to w[k+1]), face offsets off[k] = nrm[k].w[k], edge lengths. */
typedef struct { int cnt; vec2 w[MAX_VERTS], nrm[MAX_VERTS]; real off[MAX_VERTS], len[MAX_VERTS]; } wpoly;

/* Polygon-circle.  For every edge the centre is projected on the edge and the
 * parameter clamped to the edge's extent (the paper's "clipped to perpendicular
 * lines extending from both corners"); the closest of these points is q.
 * Outside the polygon: n = (c - q)/|c - q|, pen = r - |c - q|, p = q.  The
 * printed penetration formula is garbled; this is the reading that makes the
 * manifold continuous with the circle-circle one.  Centre inside the polygon
 * (paper silent): the edge of largest signed distance s <= 0 gives n = its
 * normal, pen = r - s, p = the centre projected on that edge line. */
static void manifold_pc(const wpoly *A, vec2 c, real r, manifold *m) {
    real maxsep = RC(0), mind2 = RC(0);
    int kmax = -1, kmin = -1;
    vec2 qmin = {0, 0}, dqmin = {0, 0};
    for (int k = 0; k < A->cnt; ++k) {
        real sep = dot2(A->nrm[k], c) - A->off[k];
        vec2 tau = perp2(A->nrm[k]);
        vec2 dv = sub2(c, A->w[k]);
        real s = dot2(tau, dv);
        s = rmax(rmin(s, A->len[k]), RC(0));
        vec2 q = { R_FMA(s, tau.x, A->w[k].x), R_FMA(s, tau.y, A->w[k].y) };
        vec2 dq = sub2(c, q);
        real d2 = dot2(dq, dq);
        if (kmax < 0 || sep > maxsep) { maxsep = sep; kmax = k; }
        if (kmin < 0 || d2 < mind2) { mind2 = d2; kmin = k; qmin = q; dqmin = dq; }
    }
    if (maxsep > RC(0)) {
        real d = R_SQRT(mind2);
        vec2 n;
        if (d < RC(1e-9)) n = A->nrm[kmin];
        else { real inv = RC(1) / d; n.x = dqmin.x * inv; n.y = dqmin.y * inv; }
        m->n = n; m->pen = r - d; m->p = qmin;
    } else {
        vec2 n = A->nrm[kmax];
        m->n = n; m->pen = r - maxsep;
        m->p.x = R_FMA(-maxsep, n.x, c.x);
        m->p.y = R_FMA(-maxsep, n.y, c.y);
    }
    m->active = m->pen > RC(0);
}

/* largest over the edges of X of the smallest signed distance of Y's vertices
 * to that edge line (the separating-axis search over X's edge normals). */
static real max_separation(const wpoly *X, const wpoly *Y, int *edge) {
    real best = RC(0); int bi = -1;
    for (int i = 0; i < X->cnt; ++i) {
        real lo = dot2(X->nrm[i], Y->w[0]);
        for (int j = 1; j < Y->cnt; ++j) lo = rmin(lo, dot2(X->nrm[i], Y->w[j]));
        real sep = lo - X->off[i];
        if (bi < 0 || sep > best) { best = sep; bi = i; }
    }
    *edge = bi;
    return best;
}

/* Polygon-polygon: separating-axis test over both edge-normal sets; the axis
 * of least penetration gives the reference face (on A unless B's best axis is
 * better by more than face_tol, so a resting box does not flip faces); the
 * incident face is the other polygon's edge most anti-parallel to the
 * reference normal; its two end points are clipped to the reference face's
 * side lines and each gives a manifold if it lies below the reference face.
 * m[0], m[1] follow the order of the incident edge's end points. */
static void manifold_pp(const wpoly *A, const wpoly *B, real face_tol, manifold m[2]) {
    m[0].active = m[1].active = 0;
    m[0].pen = m[1].pen = RC(-1);
    m[0].p.x = m[0].p.y = m[1].p.x = m[1].p.y = RC(0);
    m[0].n.x = m[1].n.x = RC(0); m[0].n.y = m[1].n.y = RC(1);
    int ea, eb;
    real sa = max_separation(A, B, &ea);
    real sb = max_separation(B, A, &eb);
    if (sa > RC(0) || sb > RC(0)) return;
    int ref_on_b = sb > sa + face_tol;
    const wpoly *R = ref_on_b ? B : A, *I = ref_on_b ? A : B;
    int e = ref_on_b ? eb : ea;
    vec2 n = R->nrm[e];
    vec2 v1 = R->w[e], v2 = R->w[(e + 1) % R->cnt];
    int f = 0; real fd = dot2(I->nrm[0], n);
    for (int k = 1; k < I->cnt; ++k) { real d = dot2(I->nrm[k], n); if (d < fd) { fd = d; f = k; } }
    vec2 ip[2] = { I->w[f], I->w[(f + 1) % I->cnt] };
    vec2 tau = perp2(n);
    real lo = dot2(tau, v1), hi = dot2(tau, v2);
    real s[2] = { dot2(tau, ip[0]), dot2(tau, ip[1]) };
    if ((s[0] < lo && s[1] < lo) || (s[0] > hi && s[1] > hi)) return;
    vec2 cp[2];
    for (int k = 0; k < 2; ++k) {
        cp[k] = ip[k];
        real bound = lo;
        int clip = 0;
        if (s[k] < lo) { bound = lo; clip = 1; }
        else if (s[k] > hi) { bound = hi; clip = 1; }
        if (clip) {
            real t = (bound - s[k]) / (s[1 - k] - s[k]);
            cp[k].x = R_FMA(t, ip[1 - k].x - ip[k].x, ip[k].x);
            cp[k].y = R_FMA(t, ip[1 - k].y - ip[k].y, ip[k].y);
        }
    }
    vec2 nn = n;
    if (ref_on_b) { nn.x = -n.x; nn.y = -n.y; }
    for (int k = 0; k < 2; ++k) {
        m[k].pen = R->off[e] - dot2(n, cp[k]);
        m[k].p = cp[k];
        m[k].n = nn;
        m[k].active = m[k].pen > RC(0);
    }
}

/* entry points for the geometry pins: raw world-frame inputs */
static void make_wpoly(const real *verts, int cnt, wpoly *W) {
    W->cnt = cnt;
    for (int k = 0; k < cnt; ++k) { W->w[k].x = verts[2 * k]; W->w[k].y = verts[2 * k + 1]; }
    for (int k = 0; k < cnt; ++k) {
        vec2 e = sub2(W->w[(k + 1) % cnt], W->w[k]);
        double len = sqrt((double)e.x * e.x + (double)e.y * e.y);
        W->len[k] = (real)len;
        W->nrm[k].x = (real)(e.y / len); W->nrm[k].y = (real)(-e.x / len);
        W->off[k] = dot2(W->nrm[k], W->w[k]);
    }
}
void k2d_ref_manifold_cc(const real *pa, real ra, const real *pb, real rb, real *out6) {
    manifold m; vec2 a = { pa[0], pa[1] }, b = { pb[0], pb[1] };
    manifold_cc(a, ra, b, rb, &m);
    out6[0] = m.p.x; out6[1] = m.p.y; out6[2] = m.n.x; out6[3] = m.n.y; out6[4] = m.pen; out6[5] = (real)m.active;
}
void k2d_ref_manifold_pc(const real *verts, int cnt, const real *c, real r, real *out6) {
    wpoly A; manifold m; vec2 cc = { c[0], c[1] };
    make_wpoly(verts, cnt, &A);
    manifold_pc(&A, cc, r, &m);
    out6[0] = m.p.x; out6[1] = m.p.y; out6[2] = m.n.x; out6[3] = m.n.y; out6[4] = m.pen; out6[5] = (real)m.active;
}
void k2d_ref_manifold_pp(const real *va, int ca, const real *vb, int cb, real face_tol, real *out12) {
    wpoly A, B; manifold m[2];
    make_wpoly(va, ca, &A); make_wpoly(vb, cb, &B);
    manifold_pp(&A, &B, face_tol, m);
    for (int k = 0; k < 2; ++k) {
        real *o = out12 + 6 * k;
        o[0] = m[k].p.x; o[1] = m[k].p.y; o[2] = m[k].n.x; o[3] = m[k].n.y; o[4] = m[k].pen; o[5] = (real)m[k].active;
    }
}

/* ---- level build: mass properties and per-level constants ----
 * Paper names mass, inertia and density only; the textbook formulas are used,
 * evaluated in double and rounded once: area = 1/2 sum cross(v_k, v_k+1),
 * m = density * area, I = density/12 * sum cross_k (v_k.v_k + v_k.v_k+1 +
 * v_k+1.v_k+1) about the body origin (the centroid); circle m = density pi r^2,
 * I = m r^2 / 2.  Fixated shapes have infinite mass: both inverses are 0. */
static void derive_level(ref_sim *S, int l) {
    int P = S->P, C = S->C, N = S->N;
    for (int i = 0; i < P; ++i) {
        const real *v = S->lv_verts + ((size_t)(l * P + i) * MAX_VERTS) * 2;
        int cnt = S->lv_nverts[l * P + i];
        double area2 = 0.0, second = 0.0;
        for (int k = 0; k < cnt; ++k) {
            double x0 = v[2 * k], y0 = v[2 * k + 1];
            double x1 = v[2 * ((k + 1) % cnt)], y1 = v[2 * ((k + 1) % cnt) + 1];
            double cr = x0 * y1 - y0 * x1;
            area2 += cr;
            second += cr * ((x0 * x0 + y0 * y0) + (x0 * x1 + y0 * y1) + (x1 * x1 + y1 * y1));
            double ex = x1 - x0, ey = y1 - y0;
            double len = sqrt(ex * ex + ey * ey);
            real *nr = S->lv_normals + ((size_t)(l * P + i) * MAX_VERTS + k) * 2;
            nr[0] = (real)(ey / len); nr[1] = (real)(-ex / len);
            S->lv_edge_len[(size_t)(l * P + i) * MAX_VERTS + k] = (real)len;
        }
        double rho = S->lv_density[l * N + i];
        double mass = rho * (0.5 * area2);
        double inertia = rho * (second / 12.0);
        int st = S->lv_static[l * N + i];
        S->lv_inv_mass[l * N + i] = st ? RC(0) : (real)(1.0 / mass);
        S->lv_inv_inertia[l * N + i] = st ? RC(0) : (real)(1.0 / inertia);
    }
    for (int c = 0; c < C; ++c) {
        int i = P + c;
        double r = S->lv_radius[l * C + c], rho = S->lv_density[l * N + i];
        double mass = rho * (3.14159265358979323846 * (r * r));
        double inertia = (mass * (r * r)) * 0.5;
        int st = S->lv_static[l * N + i];
        S->lv_inv_mass[l * N + i] = st ? RC(0) : (real)(1.0 / mass);
        S->lv_inv_inertia[l * N + i] = st ? RC(0) : (real)(1.0 / inertia);
    }
    for (int t = 0; t < S->T; ++t) {
        double phi = S->lv_thr_rot[l * S->T + t];
        S->lv_thr_dir[(size_t)(l * S->T + t) * 2 + 0] = (real)cos(phi);
        S->lv_thr_dir[(size_t)(l * S->T + t) * 2 + 1] = (real)sin(phi);
    }
    /* which pairs may collide: both shapes active, not both fixated, and not
     * joined by an active joint (the paper disables collision of joined shapes) */
    for (int p = 0; p < S->n_pairs; ++p) {
        int a = S->pair_a[p], b = S->pair_b[p];
        int ok = S->lv_active[l * N + a] && S->lv_active[l * N + b] &&
                 !(S->lv_static[l * N + a] && S->lv_static[l * N + b]);
        for (int j = 0; j < S->J && ok; ++j) {
            if (!S->lv_joint_active[l * S->J + j]) continue;
            int ja = S->lv_joint_a[l * S->J + j], jb = S->lv_joint_b[l * S->J + j];
            if ((ja == a && jb == b) || (ja == b && jb == a)) ok = 0;
        }
        S->lv_collide[(size_t)l * S->n_pairs + p] = (uint8_t)ok;
    }
}

#define COPY_ARR(dst, src, count, type) do { \
    (dst) = (type *)malloc(sizeof(type) * (size_t)((count) > 0 ? (count) : 1)); \
    if ((count) > 0) memcpy((dst), (src), sizeof(type) * (size_t)(count)); } while (0)
#define NEW_ARR(dst, count, type) (dst) = (type *)calloc((size_t)((count) > 0 ? (count) : 1), sizeof(type))

static void reset_env(ref_sim *S, int e, int level) {
    int N = S->N;
    memcpy(S->pos + (size_t)e * N * 2, S->lv_pos + (size_t)level * N * 2, sizeof(real) * N * 2);
    memcpy(S->vel + (size_t)e * N * 2, S->lv_vel + (size_t)level * N * 2, sizeof(real) * N * 2);
    memcpy(S->angle + (size_t)e * N, S->lv_angle + (size_t)level * N, sizeof(real) * N);
    memcpy(S->angvel + (size_t)e * N, S->lv_angvel + (size_t)level * N, sizeof(real) * N);
    memset(S->acc + (size_t)e * S->n_slots * 2, 0, sizeof(real) * S->n_slots * 2);
    memset(S->jacc + (size_t)e * S->J * 3, 0, sizeof(real) * S->J * 3);
    S->step_count[e] = 0;
    S->level_id[e] = level;
    S->status[e] = 0;
}

ref_sim *k2d_ref_create(const ref_config *cfg, const ref_levels *L) {
    ref_sim *S = (ref_sim *)calloc(1, sizeof(ref_sim));
    S->cfg = *cfg;
    int P = S->P = cfg->n_polygons, C = S->C = cfg->n_circles, N = S->N = P + C;
    int J = S->J = cfg->n_joints, T = S->T = cfg->n_thrusters, nl = cfg->n_levels, E = cfg->n_envs;
    S->n_pp = P * (P - 1) / 2; S->n_pc = P * C; S->n_cc = C * (C - 1) / 2;
    S->n_pairs = S->n_pp + S->n_pc + S->n_cc;
    S->n_slots = 2 * S->n_pp + S->n_pc + S->n_cc;
    NEW_ARR(S->pair_a, S->n_pairs, int); NEW_ARR(S->pair_b, S->n_pairs, int); NEW_ARR(S->pair_slot, S->n_pairs, int);
    /* canonical pair order: polygon-polygon (i<j), polygon-circle (polygon
     * major), circle-circle (i<j); polygon-polygon pairs own two slots. */
    int p = 0, slot = 0;
    for (int i = 0; i < P; ++i) for (int j = i + 1; j < P; ++j) { S->pair_a[p] = i; S->pair_b[p] = j; S->pair_slot[p] = slot; slot += 2; ++p; }
    for (int i = 0; i < P; ++i) for (int c = 0; c < C; ++c) { S->pair_a[p] = i; S->pair_b[p] = P + c; S->pair_slot[p] = slot; slot += 1; ++p; }
    for (int i = 0; i < C; ++i) for (int j = i + 1; j < C; ++j) { S->pair_a[p] = P + i; S->pair_b[p] = P + j; S->pair_slot[p] = slot; slot += 1; ++p; }

    COPY_ARR(S->lv_verts, L->poly_verts, nl * P * MAX_VERTS * 2, real);
    COPY_ARR(S->lv_nverts, L->poly_nverts, nl * P, int32_t);
    COPY_ARR(S->lv_radius, L->circle_radius, nl * C, real);
    COPY_ARR(S->lv_pos, L->pos, nl * N * 2, real);
    COPY_ARR(S->lv_angle, L->angle, nl * N, real);
    COPY_ARR(S->lv_vel, L->vel, nl * N * 2, real);
    COPY_ARR(S->lv_angvel, L->angvel, nl * N, real);
    COPY_ARR(S->lv_density, L->density, nl * N, real);
    COPY_ARR(S->lv_friction, L->friction, nl * N, real);
    COPY_ARR(S->lv_restitution, L->restitution, nl * N, real);
    COPY_ARR(S->lv_static, L->is_static, nl * N, int32_t);
    COPY_ARR(S->lv_role, L->role, nl * N, int32_t);
    COPY_ARR(S->lv_active, L->active, nl * N, int32_t);
    COPY_ARR(S->lv_joint_a, L->joint_a, nl * J, int32_t);
    COPY_ARR(S->lv_joint_b, L->joint_b, nl * J, int32_t);
    COPY_ARR(S->lv_anchor_a, L->joint_anchor_a, nl * J * 2, real);
    COPY_ARR(S->lv_anchor_b, L->joint_anchor_b, nl * J * 2, real);
    COPY_ARR(S->lv_motor_speed, L->motor_speed, nl * J, real);
    COPY_ARR(S->lv_motor_power, L->motor_power, nl * J, real);
    COPY_ARR(S->lv_motor_binding, L->motor_binding, nl * J, int32_t);
    COPY_ARR(S->lv_joint_active, L->joint_active, nl * J, int32_t);
    COPY_ARR(S->lv_joint_fixed, L->joint_fixed, nl * J, int32_t);
    COPY_ARR(S->lv_joint_limited, L->joint_limited, nl * J, int32_t);
    COPY_ARR(S->lv_fixed_angle, L->joint_fixed_angle, nl * J, real);
    COPY_ARR(S->lv_joint_min, L->joint_min, nl * J, real);
    COPY_ARR(S->lv_joint_max, L->joint_max, nl * J, real);
    COPY_ARR(S->lv_thr_shape, L->thr_shape, nl * T, int32_t);
    COPY_ARR(S->lv_thr_pos, L->thr_pos, nl * T * 2, real);
    COPY_ARR(S->lv_thr_rot, L->thr_rot, nl * T, real);
    COPY_ARR(S->lv_thr_power, L->thr_power, nl * T, real);
    COPY_ARR(S->lv_thr_binding, L->thr_binding, nl * T, int32_t);
    COPY_ARR(S->lv_thr_active, L->thr_active, nl * T, int32_t);
    NEW_ARR(S->lv_normals, nl * P * MAX_VERTS * 2, real);
    NEW_ARR(S->lv_edge_len, nl * P * MAX_VERTS, real);
    NEW_ARR(S->lv_inv_mass, nl * N, real);
    NEW_ARR(S->lv_inv_inertia, nl * N, real);
    NEW_ARR(S->lv_thr_dir, nl * T * 2, real);
    NEW_ARR(S->lv_collide, (size_t)nl * S->n_pairs, uint8_t);
    /* fixated shapes never move: their level velocities are forced to zero */
    for (int l = 0; l < nl; ++l) for (int i = 0; i < N; ++i) if (S->lv_static[l * N + i]) {
        S->lv_vel[(size_t)(l * N + i) * 2] = S->lv_vel[(size_t)(l * N + i) * 2 + 1] = RC(0);
        S->lv_angvel[l * N + i] = RC(0);
    }
    for (int l = 0; l < nl; ++l) derive_level(S, l);

    NEW_ARR(S->pos, (size_t)E * N * 2, real); NEW_ARR(S->vel, (size_t)E * N * 2, real);
    NEW_ARR(S->angle, (size_t)E * N, real); NEW_ARR(S->angvel, (size_t)E * N, real);
    NEW_ARR(S->acc, (size_t)E * S->n_slots * 2, real); NEW_ARR(S->jacc, (size_t)E * J * 3, real);
    NEW_ARR(S->step_count, E, int32_t); NEW_ARR(S->episode_count, E, int32_t);
    NEW_ARR(S->level_id, E, int32_t); NEW_ARR(S->status, E, int32_t);
    NEW_ARR(S->manifold, (size_t)E * S->n_slots * 6, real);
    NEW_ARR(S->counters, 8, int64_t);
    for (int e = 0; e < E; ++e) { reset_env(S, e, e % nl); S->episode_count[e] = 0; }
    return S;
}

void k2d_ref_destroy(ref_sim *S) {
    if (!S) return;
    void *ptrs[] = { S->pair_a, S->pair_b, S->pair_slot, S->lv_verts, S->lv_normals, S->lv_edge_len, S->lv_nverts,
        S->lv_radius, S->lv_pos, S->lv_angle, S->lv_vel, S->lv_angvel, S->lv_density, S->lv_friction,
        S->lv_restitution, S->lv_inv_mass, S->lv_inv_inertia, S->lv_static, S->lv_role, S->lv_active,
        S->lv_joint_a, S->lv_joint_b, S->lv_motor_binding, S->lv_joint_active, S->lv_anchor_a, S->lv_anchor_b,
        S->lv_motor_speed, S->lv_motor_power, S->lv_thr_shape, S->lv_thr_binding, S->lv_thr_active, S->lv_thr_pos,
        S->lv_thr_rot, S->lv_thr_dir, S->lv_thr_power, S->lv_collide, S->pos, S->angle, S->vel, S->angvel, S->acc,
        S->jacc, S->lv_joint_fixed, S->lv_joint_limited, S->lv_fixed_angle, S->lv_joint_min, S->lv_joint_max, S->step_count, S->episode_count, S->level_id, S->status, S->manifold, S->counters };
    for (size_t i = 0; i < sizeof(ptrs) / sizeof(ptrs[0]); ++i) free(ptrs[i]);
    free(S);
}

/* explicit reset: env e restarts on level ids[e] (or e mod n_levels), episode 0 */
void k2d_ref_reset(ref_sim *S, const int32_t *ids) {
    for (int e = 0; e < S->cfg.n_envs; ++e) {
        reset_env(S, e, ids ? ids[e] : e % S->cfg.n_levels);
        S->episode_count[e] = 0;
    }
    memset(S->counters, 0, sizeof(int64_t) * 8);
}

void k2d_ref_views(ref_sim *S, ref_views *V) {
    V->pos = S->pos; V->angle = S->angle; V->vel = S->vel; V->angvel = S->angvel; V->acc = S->acc; V->jacc = S->jacc;
    V->step_count = S->step_count; V->episode_count = S->episode_count; V->level_id = S->level_id; V->status = S->status;
    V->manifold = S->manifold; V->inv_mass = S->lv_inv_mass; V->inv_inertia = S->lv_inv_inertia;
    V->pair_a = S->pair_a; V->pair_b = S->pair_b; V->pair_slot = S->pair_slot; V->collide = S->lv_collide;
    V->counters = S->counters; V->n_pairs = S->n_pairs; V->n_slots = S->n_slots;
}

/* ---- one contact row's constants, built once per step ("pre-step") ---- */
typedef struct {
    int a, b, slot;
    vec2 n, t;
    real rn_a, rn_b, rt_a, rt_b;     /* r x n, r x t levers                     */
    real wn_a, wn_b, wt_a, wt_b;     /* inverse inertia times lever             */
    real mass_n, mass_t;             /* 1 / effective inverse mass              */
    real target, mu, corr;
} contact_row;

/* impulse of magnitude d along dir at the contact: v += j/m, w += (r x j)/I on
 * b and the opposite on a (paper: "Impulse Resolution") */
static void apply_row(real *va, real *wa, real *vb, real *wb, real ma, real mb,
                      real d, vec2 dir, real lev_a, real lev_b) {
    real px = d * dir.x, py = d * dir.y;
    va[0] = R_FMA(-ma, px, va[0]); va[1] = R_FMA(-ma, py, va[1]);
    *wa = R_FMA(-lev_a, d, *wa);
    vb[0] = R_FMA(mb, px, vb[0]); vb[1] = R_FMA(mb, py, vb[1]);
    *wb = R_FMA(lev_b, d, *wb);
}
/* relative velocity of the contact point of b with respect to a along dir:
 * dir.(vb + wb x rb - va - wa x ra) = dir.(vb - va) + wb (rb x dir) - wa (ra x dir) */
static real rel_vel(const real *va, real wa, const real *vb, real wb, vec2 dir, real r_a, real r_b) {
    vec2 dv = { vb[0] - va[0], vb[1] - va[1] };
    real v = dot2(dir, dv);
    v = R_FMA(wb, r_b, v);
    v = R_FMA(-wa, r_a, v);
    return v;
}

typedef struct {
    int a, b, on;
    vec2 ra, rb, bias, corr_dir;
    real i11, i12, i22;              /* inverse of the 2x2 effective mass matrix */
    real ma, mb, ia, ib;
    /* angular row (paper, "Fixed Joints" and "Joint Limits"): 0 none, 1 fixed, 2 beyond the upper limit, 3 beyond the lower */
    int ang;
    real kr, bias_r;                 /* 1 / (1/I_a + 1/I_b); gamma * angular error */
} joint_row;

static void step_env(ref_sim *S, int e, const real *act, real *out_reward, uint8_t *out_done, int64_t *cnt) {
    const ref_config *cf = &S->cfg;
    const int P = S->P, C = S->C, N = S->N, J = S->J, T = S->T;
    real *pos = S->pos + (size_t)e * N * 2, *vel = S->vel + (size_t)e * N * 2;
    real *ang = S->angle + (size_t)e * N, *angvel = S->angvel + (size_t)e * N;
    real *acc = S->acc + (size_t)e * S->n_slots * 2, *jacc = S->jacc + (size_t)e * J * 3;
    real *trace = S->manifold + (size_t)e * S->n_slots * 6;

    /* a frozen env (non-finite state, no auto-reset) reports done and nothing else */
    if (S->status[e] & STATUS_NONFINITE) { *out_reward = RC(0); *out_done = 1; return; }

    const int l = S->level_id[e];
    const real *inv_mass = S->lv_inv_mass + (size_t)l * N, *inv_inertia = S->lv_inv_inertia + (size_t)l * N;
    const real *fric = S->lv_friction + (size_t)l * N, *rest = S->lv_restitution + (size_t)l * N;
    const int32_t *active = S->lv_active + (size_t)l * N, *role = S->lv_role + (size_t)l * N;
    const uint8_t *collide = S->lv_collide + (size_t)l * S->n_pairs;
    const real dt = cf->dt;

    /* distance between the first green and the first blue shape before the step (dense reward) */
    int dense_g = -1, dense_b = -1;
    real dense_d0 = RC(0);
    if (cf->dense_kappa != RC(0)) {
        for (int i = N - 1; i >= 0; --i) if (active[i]) { if (role[i] == ROLE_GREEN) dense_g = i; if (role[i] == ROLE_BLUE) dense_b = i; }
        if (dense_g >= 0 && dense_b >= 0) {
            vec2 dd = { pos[2 * dense_b] - pos[2 * dense_g], pos[2 * dense_b + 1] - pos[2 * dense_g + 1] };
            dense_d0 = R_SQRT(dot2(dd, dd));
        }
    }

    /* Alg. 1 line 2: gravity on movable shapes */
    const real gdt = cf->gravity_y * dt;
    for (int i = 0; i < N; ++i)
        if (active[i] && inv_mass[i] > RC(0)) vel[2 * i + 1] = vel[2 * i + 1] + gdt;

    /* world-frame geometry from the poses at the start of the step */
    real cs[32], sn[32];
    wpoly W[16];
    real bb[32][4]; /* minx, miny, maxx, maxy */
    for (int i = 0; i < N; ++i) k2d_ref_sincos(ang[i], &cs[i], &sn[i]);
    for (int i = 0; i < P; ++i) {
        wpoly *w = &W[i];
        w->cnt = S->lv_nverts[l * P + i];
        const real *lv = S->lv_verts + ((size_t)(l * P + i) * MAX_VERTS) * 2;
        const real *ln = S->lv_normals + ((size_t)(l * P + i) * MAX_VERTS) * 2;
        for (int k = 0; k < w->cnt; ++k) {
            vec2 loc = { lv[2 * k], lv[2 * k + 1] }, nl = { ln[2 * k], ln[2 * k + 1] };
            vec2 r = rot2(cs[i], sn[i], loc);
            w->w[k].x = r.x + pos[2 * i]; w->w[k].y = r.y + pos[2 * i + 1];
            w->nrm[k] = rot2(cs[i], sn[i], nl);
            w->off[k] = dot2(w->nrm[k], w->w[k]);
            w->len[k] = S->lv_edge_len[(size_t)(l * P + i) * MAX_VERTS + k];
        }
        bb[i][0] = bb[i][2] = w->w[0].x; bb[i][1] = bb[i][3] = w->w[0].y;
        for (int k = 1; k < w->cnt; ++k) {
            bb[i][0] = rmin(bb[i][0], w->w[k].x); bb[i][1] = rmin(bb[i][1], w->w[k].y);
            bb[i][2] = rmax(bb[i][2], w->w[k].x); bb[i][3] = rmax(bb[i][3], w->w[k].y);
        }
    }
    for (int c = 0; c < C; ++c) {
        int i = P + c; real r = S->lv_radius[l * C + c];
        bb[i][0] = pos[2 * i] - r; bb[i][1] = pos[2 * i + 1] - r;
        bb[i][2] = pos[2 * i] + r; bb[i][3] = pos[2 * i + 1] + r;
    }

    /* Alg. 1 line 3: manifolds for every pair that may collide, canonical order.
     * The box test in front is part of the specified step, not an optimisation
     * the results may depend on: boxes further apart than aabb_margin cannot
     * hold an active manifold (a test runs the oracle with it off to show so). */
    manifold man[256];
    int touch_gb = 0, touch_gr = 0;
    for (int s = 0; s < S->n_slots; ++s) { man[s].active = 0; man[s].pen = RC(-1); man[s].p.x = man[s].p.y = RC(0); man[s].n.x = RC(0); man[s].n.y = RC(1); }
    for (int p = 0; p < S->n_pairs; ++p) {
        if (!collide[p]) continue;
        int a = S->pair_a[p], b = S->pair_b[p], s = S->pair_slot[p];
        if (cf->broadphase) {
            real mg = cf->aabb_margin;
            if (bb[a][2] + mg < bb[b][0] || bb[b][2] + mg < bb[a][0] ||
                bb[a][3] + mg < bb[b][1] || bb[b][3] + mg < bb[a][1]) continue;
        }
        vec2 pa = { pos[2 * a], pos[2 * a + 1] }, pb = { pos[2 * b], pos[2 * b + 1] };
        int any;
        cnt[4 + (b < P ? 0 : (a < P ? 1 : 2))] += 1;
        if (b < P) { manifold_pp(&W[a], &W[b], cf->face_tol, &man[s]); any = man[s].active || man[s + 1].active; }
        else if (a < P) { manifold_pc(&W[a], pb, S->lv_radius[l * C + (b - P)], &man[s]); any = man[s].active; }
        else { manifold_cc(pa, S->lv_radius[l * C + (a - P)], pb, S->lv_radius[l * C + (b - P)], &man[s]); any = man[s].active; }
        /* touch flags of this step: an active manifold between green and blue / green and red */
        if (any) {
            cnt[7] += 1;
            int r1 = role[a], r2 = role[b];
            if ((r1 == ROLE_GREEN && r2 == ROLE_BLUE) || (r1 == ROLE_BLUE && r2 == ROLE_GREEN)) touch_gb = 1;
            if ((r1 == ROLE_GREEN && r2 == ROLE_RED) || (r1 == ROLE_RED && r2 == ROLE_GREEN)) touch_gr = 1;
        }
    }
    for (int s = 0; s < S->n_slots; ++s) {
        real *t = trace + 6 * s;
        t[0] = man[s].p.x; t[1] = man[s].p.y; t[2] = man[s].n.x; t[3] = man[s].n.y; t[4] = man[s].pen; t[5] = (real)man[s].active;
    }

    /* Alg. 1 line 4: motors.  j_r = p tanh((wa - wb - s A) rho), a true impulse
     * applied once; a loses j_r / I_a and b gains j_r / I_b so that wa - wb is
     * driven towards s A.  A = action clipped to [-1, 1]. */
    for (int j = 0; j < J; ++j) {
        int a = S->lv_joint_a[l * J + j], b = S->lv_joint_b[l * J + j];
        if (!(S->lv_joint_active[l * J + j] && active[a] && active[b] && (inv_mass[a] + inv_mass[b] > RC(0)))) continue;
        /* "Action Space": continuous in [-1, 1]; multi-discrete 0 = off, 1 = forwards, 2 = backwards at full power */
        real av = act[S->lv_motor_binding[l * J + j]];
        real A = cf->discrete_actions ? (av == RC(1) ? RC(1) : (av == RC(2) ? RC(-1) : RC(0))) : rmax(rmin(av, RC(1)), RC(-1));
        real d = angvel[a] - angvel[b];
        real arg = R_FMA(-S->lv_motor_speed[l * J + j], A, d) * cf->motor_rho;
        real jr = S->lv_motor_power[l * J + j] * k2d_ref_tanh(arg);
        angvel[a] = R_FMA(-jr, inv_inertia[a], angvel[a]);
        angvel[b] = R_FMA(jr, inv_inertia[b], angvel[b]);
    }
    /* Alg. 1 line 5: thrusters.  Force p A along the facing direction at the
     * attachment point, turned into the impulse p A dt.  A clipped to [0, 1]. */
    for (int t = 0; t < T; ++t) {
        if (!S->lv_thr_active[l * T + t]) continue;
        int i = S->lv_thr_shape[l * T + t];
        if (!active[i]) continue;
        /* continuous in [0, 1]; multi-discrete 0 = off, anything else = full power */
        real tv = act[S->lv_thr_binding[l * T + t]];
        real A = cf->discrete_actions ? (tv != RC(0) ? RC(1) : RC(0)) : rmax(rmin(tv, RC(1)), RC(0));
        vec2 ld = { S->lv_thr_dir[(size_t)(l * T + t) * 2], S->lv_thr_dir[(size_t)(l * T + t) * 2 + 1] };
        vec2 lp = { S->lv_thr_pos[(size_t)(l * T + t) * 2], S->lv_thr_pos[(size_t)(l * T + t) * 2 + 1] };
        vec2 dir = rot2(cs[i], sn[i], ld), r = rot2(cs[i], sn[i], lp);
        real imp = (S->lv_thr_power[l * T + t] * A) * dt;
        vec2 jv = { imp * dir.x, imp * dir.y };
        vel[2 * i] = R_FMA(jv.x, inv_mass[i], vel[2 * i]);
        vel[2 * i + 1] = R_FMA(jv.y, inv_mass[i], vel[2 * i + 1]);
        angvel[i] = R_FMA(cross2(r, jv), inv_inertia[i], angvel[i]);
    }

    /* contact rows for the active manifolds, canonical order */
    contact_row rows[256];
    int n_rows = 0;
    for (int p = 0; p < S->n_pairs; ++p) {
        int a = S->pair_a[p], b = S->pair_b[p];
        int nslot = (b < P) ? 2 : 1;
        for (int k = 0; k < nslot; ++k) {
            int s = S->pair_slot[p] + k;
            if (!man[s].active) { acc[2 * s] = acc[2 * s + 1] = RC(0); continue; } /* paper: impulses wiped when not colliding */
            if (!cf->warm_start) acc[2 * s] = acc[2 * s + 1] = RC(0);
            contact_row *r = &rows[n_rows++];
            r->a = a; r->b = b; r->slot = s;
            r->n = man[s].n; r->t = perp2(man[s].n);
            vec2 xa = { pos[2 * a], pos[2 * a + 1] }, xb = { pos[2 * b], pos[2 * b + 1] };
            vec2 ra = sub2(man[s].p, xa), rb = sub2(man[s].p, xb);
            real ma = inv_mass[a], mb = inv_mass[b], ia = inv_inertia[a], ib = inv_inertia[b];
            r->rn_a = cross2(ra, r->n); r->rn_b = cross2(rb, r->n);
            r->rt_a = cross2(ra, r->t); r->rt_b = cross2(rb, r->t);
            r->wn_a = ia * r->rn_a; r->wn_b = ib * r->rn_b;
            r->wt_a = ia * r->rt_a; r->wt_b = ib * r->rt_b;
            /* denominator of the paper's impulse equation */
            real kn = ma + mb; kn = R_FMA(r->wn_a, r->rn_a, kn); kn = R_FMA(r->wn_b, r->rn_b, kn);
            real kt = ma + mb; kt = R_FMA(r->wt_a, r->rt_a, kt); kt = R_FMA(r->wt_b, r->rt_b, kt);
            r->mass_n = RC(1) / kn; r->mass_t = RC(1) / kt;
            /* combination rules: e = min, mu = sqrt(mu_a^2 + mu_b^2) */
            real er = rmin(rest[a], rest[b]);
            r->mu = R_SQRT(R_FMA(fric[a], fric[a], fric[b] * fric[b]));
            /* target normal velocity: -e v_n0 for an approach faster than the
             * threshold (measured now, before warm starting), plus the velocity
             * correction alpha * penetration beyond the slop */
            real vn0 = rel_vel(vel + 2 * a, angvel[a], vel + 2 * b, angvel[b], r->n, r->rn_a, r->rn_b);
            real depth = rmax(man[s].pen - cf->slop, RC(0));
            real bounce = (vn0 < -cf->restitution_threshold) ? (-er * vn0) : RC(0);
            r->target = bounce + cf->contact_alpha * depth;
            r->corr = (cf->contact_beta * depth) / (ma + mb);
        }
    }
    cnt[2] += n_rows;

    /* joint rows: the joined points must coincide and have no relative velocity */
    joint_row jr[16];
    for (int j = 0; j < J; ++j) {
        joint_row *q = &jr[j];
        int a = S->lv_joint_a[l * J + j], b = S->lv_joint_b[l * J + j];
        q->a = a; q->b = b;
        q->on = S->lv_joint_active[l * J + j] && active[a] && active[b] && (inv_mass[a] + inv_mass[b] > RC(0));
        q->ang = 0;
        if (!q->on) { jacc[3 * j] = jacc[3 * j + 1] = jacc[3 * j + 2] = RC(0); continue; }
        if (!cf->warm_start) jacc[3 * j] = jacc[3 * j + 1] = jacc[3 * j + 2] = RC(0);
        vec2 la = { S->lv_anchor_a[(size_t)(l * J + j) * 2], S->lv_anchor_a[(size_t)(l * J + j) * 2 + 1] };
        vec2 lb = { S->lv_anchor_b[(size_t)(l * J + j) * 2], S->lv_anchor_b[(size_t)(l * J + j) * 2 + 1] };
        q->ra = rot2(cs[a], sn[a], la); q->rb = rot2(cs[b], sn[b], lb);
        q->ma = inv_mass[a]; q->mb = inv_mass[b]; q->ia = inv_inertia[a]; q->ib = inv_inertia[b];
        vec2 gap = { (pos[2 * b] + q->rb.x) - (pos[2 * a] + q->ra.x), (pos[2 * b + 1] + q->rb.y) - (pos[2 * a + 1] + q->ra.y) };
        real msum = q->ma + q->mb;
        real k11 = msum; k11 = R_FMA(q->ia * q->ra.y, q->ra.y, k11); k11 = R_FMA(q->ib * q->rb.y, q->rb.y, k11);
        real k22 = msum; k22 = R_FMA(q->ia * q->ra.x, q->ra.x, k22); k22 = R_FMA(q->ib * q->rb.x, q->rb.x, k22);
        real k12 = -((q->ia * q->ra.x) * q->ra.y); k12 = R_FMA(-(q->ib * q->rb.x), q->rb.y, k12);
        real det = R_FMA(k11, k22, -(k12 * k12));
        real inv_det = RC(1) / det;
        q->i11 = k22 * inv_det; q->i22 = k11 * inv_det; q->i12 = -(k12 * inv_det);
        q->bias.x = cf->joint_alpha * gap.x; q->bias.y = cf->joint_alpha * gap.y;
        real share = cf->joint_beta / msum;
        q->corr_dir.x = share * gap.x; q->corr_dir.y = share * gap.y;
        /* angular row.  Fixed joint ("Fixed Joints"): the relative rotation angle_a - angle_b is held at
         * the joint's angle, error C, velocity correction gamma * C, accumulated and warm-started.
         * Limited revolute joint ("Joint Limits"): a row only while the relative rotation is beyond a
         * limit, C measured from that limit, never accumulated.  Both from the poses at the start of
         * the step, like the manifolds. */
        real isum = q->ia + q->ib;
        q->kr = RC(0); q->bias_r = RC(0);
        if (isum > RC(0)) {
            real rel = ang[a] - ang[b];
            if (S->lv_joint_fixed[l * J + j]) {
                q->ang = 1; q->kr = RC(1) / isum;
                q->bias_r = cf->joint_gamma * (rel - S->lv_fixed_angle[l * J + j]);
            } else if (S->lv_joint_limited[l * J + j]) {
                real hi = S->lv_joint_max[l * J + j], lo = S->lv_joint_min[l * J + j];
                if (rel > hi) { q->ang = 2; q->kr = RC(1) / isum; q->bias_r = cf->joint_gamma * (rel - hi); }
                else if (rel < lo) { q->ang = 3; q->kr = RC(1) / isum; q->bias_r = cf->joint_gamma * (rel - lo); }
            }
        }
        if (q->ang != 1) jacc[3 * j + 2] = RC(0);
    }

    /* Alg. 1 lines 6-9: warm start, contacts first, then joints */
    for (int i = 0; i < n_rows; ++i) {
        contact_row *r = &rows[i];
        apply_row(vel + 2 * r->a, &angvel[r->a], vel + 2 * r->b, &angvel[r->b], inv_mass[r->a], inv_mass[r->b],
                  acc[2 * r->slot], r->n, r->wn_a, r->wn_b);
        apply_row(vel + 2 * r->a, &angvel[r->a], vel + 2 * r->b, &angvel[r->b], inv_mass[r->a], inv_mass[r->b],
                  acc[2 * r->slot + 1], r->t, r->wt_a, r->wt_b);
    }
    for (int j = 0; j < J; ++j) {
        joint_row *q = &jr[j];
        if (!q->on) continue;
        vec2 lam = { jacc[3 * j], jacc[3 * j + 1] };
        real *va = vel + 2 * q->a, *vb = vel + 2 * q->b;
        va[0] = R_FMA(-q->ma, lam.x, va[0]); va[1] = R_FMA(-q->ma, lam.y, va[1]);
        angvel[q->a] = R_FMA(-q->ia, cross2(q->ra, lam), angvel[q->a]);
        vb[0] = R_FMA(q->mb, lam.x, vb[0]); vb[1] = R_FMA(q->mb, lam.y, vb[1]);
        angvel[q->b] = R_FMA(q->ib, cross2(q->rb, lam), angvel[q->b]);
        if (q->ang == 1) {
            real lr = jacc[3 * j + 2];
            angvel[q->a] = R_FMA(-lr, q->ia, angvel[q->a]);
            angvel[q->b] = R_FMA(lr, q->ib, angvel[q->b]);
        }
    }

    /* Alg. 1 lines 10-13: solver iterations, joints then contacts, sequential */
    for (int it = 0; it < cf->solver_iters; ++it) {
        for (int j = 0; j < J; ++j) {
            joint_row *q = &jr[j];
            if (!q->on) continue;
            real *va = vel + 2 * q->a, *vb = vel + 2 * q->b;
            real wa = angvel[q->a], wb = angvel[q->b];
            /* relative velocity of the joined points: vb + wb x rb - va - wa x ra */
            real cx = (R_FMA(-wb, q->rb.y, vb[0])) - (R_FMA(-wa, q->ra.y, va[0]));
            real cy = (R_FMA(wb, q->rb.x, vb[1])) - (R_FMA(wa, q->ra.x, va[1]));
            real rx = -(cx + q->bias.x), ry = -(cy + q->bias.y);
            vec2 lam = { R_FMA(q->i11, rx, q->i12 * ry), R_FMA(q->i12, rx, q->i22 * ry) };
            jacc[3 * j] = jacc[3 * j] + lam.x; jacc[3 * j + 1] = jacc[3 * j + 1] + lam.y;
            va[0] = R_FMA(-q->ma, lam.x, va[0]); va[1] = R_FMA(-q->ma, lam.y, va[1]);
            angvel[q->a] = R_FMA(-q->ia, cross2(q->ra, lam), wa);
            vb[0] = R_FMA(q->mb, lam.x, vb[0]); vb[1] = R_FMA(q->mb, lam.y, vb[1]);
            angvel[q->b] = R_FMA(q->ib, cross2(q->rb, lam), wb);
            if (q->ang) {
                /* angular impulse j_r = (w_a - w_b + correction) / (1/I_a + 1/I_b): a loses j_r / I_a, b gains j_r / I_b */
                real wrel = angvel[q->a] - angvel[q->b];
                real v;
                if (q->ang == 1) v = wrel + q->bias_r;
                else if (q->ang == 2) {
                    /* beyond the upper limit: no correction if already returning; only ever pushes back */
                    v = (wrel < RC(0)) ? wrel : wrel + q->bias_r;
                    v = rmax(v, RC(0));
                } else {
                    v = (wrel > RC(0)) ? wrel : wrel + q->bias_r;
                    v = rmin(v, RC(0));
                }
                real lr = v * q->kr;
                if (q->ang == 1) jacc[3 * j + 2] = jacc[3 * j + 2] + lr;
                angvel[q->a] = R_FMA(-lr, q->ia, angvel[q->a]);
                angvel[q->b] = R_FMA(lr, q->ib, angvel[q->b]);
            }
        }
        /* Batched impulse resolution (paper, "Parallelised Computation and Batched Impulse Resolution"): the manifold
         * slots are cut into batches of solver_batch; the rows of a batch are solved side by side, all against the
         * velocities the batch starts with, and only then applied; batches follow one another.  The active manifolds
         * are spread over as many batches as possible: the i-th active row (canonical order) goes to batch i mod
         * n_batches.  With no more active rows than batches every batch holds one row and this is the sequential
         * sweep below, operation for operation. */
        if (cf->solver_batch > 0) {
            const int n_batches = (S->n_slots + cf->solver_batch - 1) / cf->solver_batch;
            real dn[256], dtan[256];
            for (int b = 0; b < n_batches && b < n_rows; ++b) {
                for (int i = b; i < n_rows; i += n_batches) {
                    contact_row *r = &rows[i];
                    /* private copies of the two bodies' velocities: the row's friction part sees its own normal impulse, nobody else's */
                    real va[2] = { vel[2 * r->a], vel[2 * r->a + 1] }, vb[2] = { vel[2 * r->b], vel[2 * r->b + 1] };
                    real wa = angvel[r->a], wb = angvel[r->b];
                    real ma = inv_mass[r->a], mb = inv_mass[r->b];
                    real vn = rel_vel(va, wa, vb, wb, r->n, r->rn_a, r->rn_b);
                    real lam = (r->target - vn) * r->mass_n;
                    real old = acc[2 * r->slot];
                    real nw = rmax(old + lam, RC(0));
                    acc[2 * r->slot] = nw;
                    dn[i] = nw - old;
                    apply_row(va, &wa, vb, &wb, ma, mb, dn[i], r->n, r->wn_a, r->wn_b);
                    real vt = rel_vel(va, wa, vb, wb, r->t, r->rt_a, r->rt_b);
                    real lamt = (-vt) * r->mass_t;
                    real lim = r->mu * nw;
                    real oldt = acc[2 * r->slot + 1];
                    real nwt = rmax(rmin(oldt + lamt, lim), -lim);
                    acc[2 * r->slot + 1] = nwt;
                    dtan[i] = nwt - oldt;
                }
                for (int i = b; i < n_rows; i += n_batches) {
                    contact_row *r = &rows[i];
                    real ma = inv_mass[r->a], mb = inv_mass[r->b];
                    apply_row(vel + 2 * r->a, &angvel[r->a], vel + 2 * r->b, &angvel[r->b], ma, mb, dn[i], r->n, r->wn_a, r->wn_b);
                    apply_row(vel + 2 * r->a, &angvel[r->a], vel + 2 * r->b, &angvel[r->b], ma, mb, dtan[i], r->t, r->wt_a, r->wt_b);
                }
            }
            continue;
        }
        for (int i = 0; i < n_rows; ++i) {
            contact_row *r = &rows[i];
            real *va = vel + 2 * r->a, *vb = vel + 2 * r->b;
            real ma = inv_mass[r->a], mb = inv_mass[r->b];
            /* normal row: accumulated impulse kept >= 0 */
            real vn = rel_vel(va, angvel[r->a], vb, angvel[r->b], r->n, r->rn_a, r->rn_b);
            real lam = (r->target - vn) * r->mass_n;
            real old = acc[2 * r->slot];
            real nw = rmax(old + lam, RC(0));
            acc[2 * r->slot] = nw;
            apply_row(va, &angvel[r->a], vb, &angvel[r->b], ma, mb, nw - old, r->n, r->wn_a, r->wn_b);
            /* friction row: |accumulated tangent impulse| <= mu * accumulated normal impulse */
            real vt = rel_vel(va, angvel[r->a], vb, angvel[r->b], r->t, r->rt_a, r->rt_b);
            real lamt = (-vt) * r->mass_t;
            real lim = r->mu * nw;
            real oldt = acc[2 * r->slot + 1];
            real nwt = rmax(rmin(oldt + lamt, lim), -lim);
            acc[2 * r->slot + 1] = nwt;
            apply_row(va, &angvel[r->a], vb, &angvel[r->b], ma, mb, nwt - oldt, r->t, r->wt_a, r->wt_b);
        }
    }

    /* Alg. 1 line 15: Euler step with the solved velocities (semi-implicit) */
    for (int i = 0; i < N; ++i) {
        if (!active[i]) continue;
        pos[2 * i] = R_FMA(dt, vel[2 * i], pos[2 * i]);
        pos[2 * i + 1] = R_FMA(dt, vel[2 * i + 1], pos[2 * i + 1]);
        ang[i] = R_FMA(dt, angvel[i], ang[i]);
    }
    /* positional corrections (beta * penetration), contacts then joints, from
     * the start-of-step penetration and gap, translation only */
    for (int i = 0; i < n_rows; ++i) {
        contact_row *r = &rows[i];
        real ca = inv_mass[r->a] * r->corr, cb = inv_mass[r->b] * r->corr;
        pos[2 * r->a] = R_FMA(-ca, r->n.x, pos[2 * r->a]); pos[2 * r->a + 1] = R_FMA(-ca, r->n.y, pos[2 * r->a + 1]);
        pos[2 * r->b] = R_FMA(cb, r->n.x, pos[2 * r->b]); pos[2 * r->b + 1] = R_FMA(cb, r->n.y, pos[2 * r->b + 1]);
    }
    for (int j = 0; j < J; ++j) {
        joint_row *q = &jr[j];
        if (!q->on) continue;
        pos[2 * q->a] = R_FMA(q->ma, q->corr_dir.x, pos[2 * q->a]); pos[2 * q->a + 1] = R_FMA(q->ma, q->corr_dir.y, pos[2 * q->a + 1]);
        pos[2 * q->b] = R_FMA(-q->mb, q->corr_dir.x, pos[2 * q->b]); pos[2 * q->b + 1] = R_FMA(-q->mb, q->corr_dir.y, pos[2 * q->b + 1]);
    }

    /* reward and termination: green touches blue = +1, green touches red = -1 */
    int finite = 1;
    for (int i = 0; i < N; ++i)
        finite = finite && is_finite_real(pos[2 * i]) && is_finite_real(pos[2 * i + 1]) && is_finite_real(ang[i]) &&
                 is_finite_real(vel[2 * i]) && is_finite_real(vel[2 * i + 1]) && is_finite_real(angvel[i]);
    S->step_count[e] += 1;
    int timeout = cf->max_episode_steps > 0 && S->step_count[e] >= cf->max_episode_steps;
    real reward = (real)(touch_gb - touch_gr);
    /* "Reward": auxiliary dense signal kappa (d_t - d_{t+1}), d = distance between the green and the blue shape
     * (the first of each by index), before and after this step */
    if (cf->dense_kappa != RC(0) && dense_g >= 0 && dense_b >= 0) {
        vec2 dd = { pos[2 * dense_b] - pos[2 * dense_g], pos[2 * dense_b + 1] - pos[2 * dense_g + 1] };
        real d1 = R_SQRT(dot2(dd, dd));
        reward = reward + cf->dense_kappa * (dense_d0 - d1);
    }
    int done = touch_gb || touch_gr || timeout;
    if (!finite) { reward = RC(0); done = 1; S->status[e] |= STATUS_NONFINITE; cnt[0] += 1; }
    *out_reward = reward; *out_done = (uint8_t)done;
    cnt[3] += 1;

    if (done && cf->auto_reset != RESET_NONE) {
        S->episode_count[e] += 1;
        int level = l;
        if (cf->auto_reset == RESET_POOL)
            level = (int)(reset_hash(cf->seed, (uint64_t)(cf->env_offset + e), (uint64_t)S->episode_count[e]) % (uint64_t)cf->n_levels);
        reset_env(S, e, level);
        cnt[1] += 1;
    }
}

/* actions [ceil(n_steps / frame_skip)][n_envs][n_actions]: every row is held for frame_skip steps (the paper's
 * frame skip; 1 = a row per step); reward, done [n_steps][n_envs] */
static void step_range(ref_sim *S, int e0, int e1, const real *actions, int n_steps, real *reward, uint8_t *done, int64_t *cnt) {
    int E = S->cfg.n_envs, A = S->cfg.n_actions, fs = S->cfg.frame_skip > 0 ? S->cfg.frame_skip : 1;
    for (int e = e0; e < e1; ++e)
        for (int s = 0; s < n_steps; ++s)
            step_env(S, e, actions + ((size_t)(s / fs) * E + e) * A, reward + (size_t)s * E + e, done + (size_t)s * E + e, cnt);
}

typedef struct { ref_sim *S; int e0, e1, n_steps; const real *actions; real *reward; uint8_t *done; int64_t cnt[8]; } job;
static void *job_main(void *arg) {
    job *j = (job *)arg;
    step_range(j->S, j->e0, j->e1, j->actions, j->n_steps, j->reward, j->done, j->cnt);
    return NULL;
}

void k2d_ref_step(ref_sim *S, const real *actions, int n_steps, real *reward, uint8_t *done, int n_threads) {
    int E = S->cfg.n_envs;
    if (n_threads < 1) n_threads = 1;
    if (n_threads > E) n_threads = E;
    job *jobs = (job *)calloc((size_t)n_threads, sizeof(job));
    pthread_t *th = (pthread_t *)calloc((size_t)n_threads, sizeof(pthread_t));
    for (int t = 0; t < n_threads; ++t) {
        jobs[t].S = S; jobs[t].n_steps = n_steps; jobs[t].actions = actions; jobs[t].reward = reward; jobs[t].done = done;
        jobs[t].e0 = (int)((int64_t)E * t / n_threads); jobs[t].e1 = (int)((int64_t)E * (t + 1) / n_threads);
        if (n_threads > 1) pthread_create(&th[t], NULL, job_main, &jobs[t]); else job_main(&jobs[t]);
    }
    for (int t = 0; t < n_threads; ++t) {
        if (n_threads > 1) pthread_join(th[t], NULL);
        for (int k = 0; k < 8; ++k) S->counters[k] += jobs[t].cnt[k];
    }
    free(jobs); free(th);
}

/* ---- symbolic per-entity observation (paper: "Observation Spaces" tables) ----
 * shape row (29): pos 2, vel 2, inverse mass, inverse inertia, density,
 * tanh(w/10), one-hot role 4, sin, cos of rotation, friction, restitution,
 * one-hot type 2 (polygon, circle), radius, 8 body-frame vertex coordinates,
 * one-hot triangle/rectangle.  Joint rows, two per joint (from a to b, then
 * from b to a) (11 + n_actions): active, is_fixed = 0, anchor w.r.t. from 2,
 * anchor w.r.t. to 2, motor power, motor speed, motor permanently on = 0,
 * one-hot of the action binding, sin, cos of (rotation_to - rotation_from).
 * Thruster row (6): active, attachment point 2, power, sin, cos of the
 * world-frame facing angle.  Inactive entities are all zeros. */
int k2d_ref_obs_floats(const ref_config *cf) {
    int N = cf->n_polygons + cf->n_circles;
    return N * 29 + cf->n_joints * 2 * (11 + cf->n_actions) + cf->n_thrusters * 6;
}
void k2d_ref_obs(ref_sim *S, real *obs) {
    const ref_config *cf = &S->cfg;
    int P = S->P, C = S->C, N = S->N, J = S->J, T = S->T, A = cf->n_actions;
    int width = k2d_ref_obs_floats(cf);
    for (int e = 0; e < cf->n_envs; ++e) {
        real *o = obs + (size_t)e * width;
        memset(o, 0, sizeof(real) * width);
        int l = S->level_id[e];
        const real *pos = S->pos + (size_t)e * N * 2, *vel = S->vel + (size_t)e * N * 2;
        const real *ang = S->angle + (size_t)e * N, *angvel = S->angvel + (size_t)e * N;
        real cs[32], sn[32];
        for (int i = 0; i < N; ++i) k2d_ref_sincos(ang[i], &cs[i], &sn[i]);
        for (int i = 0; i < N; ++i) {
            real *r = o + i * 29;
            if (!S->lv_active[l * N + i]) continue;
            r[0] = pos[2 * i]; r[1] = pos[2 * i + 1]; r[2] = vel[2 * i]; r[3] = vel[2 * i + 1];
            r[4] = S->lv_inv_mass[l * N + i]; r[5] = S->lv_inv_inertia[l * N + i]; r[6] = S->lv_density[l * N + i];
            r[7] = k2d_ref_tanh(angvel[i] * RC(0.1));
            r[8 + S->lv_role[l * N + i]] = RC(1);
            r[12] = sn[i]; r[13] = cs[i];
            r[14] = S->lv_friction[l * N + i]; r[15] = S->lv_restitution[l * N + i];
            if (i < P) {
                r[16] = RC(1);
                int cnt = S->lv_nverts[l * P + i];
                const real *v = S->lv_verts + ((size_t)(l * P + i) * MAX_VERTS) * 2;
                for (int k = 0; k < cnt; ++k) { r[19 + 2 * k] = v[2 * k]; r[20 + 2 * k] = v[2 * k + 1]; }
                r[27 + (cnt == 4 ? 1 : 0)] = RC(1);
            } else {
                r[17] = RC(1);
                r[18] = S->lv_radius[l * C + (i - P)];
            }
        }
        int jw = 11 + A;
        for (int j = 0; j < J; ++j) {
            if (!S->lv_joint_active[l * J + j]) continue;
            int a = S->lv_joint_a[l * J + j], b = S->lv_joint_b[l * J + j];
            const real *la = S->lv_anchor_a + (size_t)(l * J + j) * 2, *lb = S->lv_anchor_b + (size_t)(l * J + j) * 2;
            for (int d = 0; d < 2; ++d) {
                real *r = o + N * 29 + (2 * j + d) * jw;
                int from = d ? b : a, to = d ? a : b;
                const real *lf = d ? lb : la, *lt = d ? la : lb;
                r[0] = RC(1); r[1] = S->lv_joint_fixed[l * J + j] ? RC(1) : RC(0);
                r[2] = lf[0]; r[3] = lf[1]; r[4] = lt[0]; r[5] = lt[1];
                r[6] = S->lv_motor_power[l * J + j]; r[7] = S->lv_motor_speed[l * J + j]; r[8] = RC(0);
                r[9 + S->lv_motor_binding[l * J + j]] = RC(1);
                /* sin, cos of (to - from) by the angle-difference identities */
                r[9 + A] = R_FMA(sn[to], cs[from], -(cs[to] * sn[from]));
                r[10 + A] = R_FMA(cs[to], cs[from], sn[to] * sn[from]);
            }
        }
        for (int t = 0; t < T; ++t) {
            if (!S->lv_thr_active[l * T + t]) continue;
            real *r = o + N * 29 + 2 * J * jw + t * 6;
            int i = S->lv_thr_shape[l * T + t];
            vec2 ld = { S->lv_thr_dir[(size_t)(l * T + t) * 2], S->lv_thr_dir[(size_t)(l * T + t) * 2 + 1] };
            vec2 d = rot2(cs[i], sn[i], ld);
            r[0] = RC(1);
            r[1] = S->lv_thr_pos[(size_t)(l * T + t) * 2]; r[2] = S->lv_thr_pos[(size_t)(l * T + t) * 2 + 1];
            r[3] = S->lv_thr_power[l * T + t];
            r[4] = d.y; r[5] = d.x;
        }
    }
}

/* ---- pixel observation ---------------------------------------------------
 * The paper gives the size only ("125 x 125 observation", section "Pixels" of
 * the network details).  Reading: an RGBA byte image per env, row 0 at the top;
 * the centre of pixel (row r, column c) is the world point
 * x = -3.125 + (c + 0.5) * 0.05, y = 5.75 - (r + 0.5) * 0.05 (a 6.25 m window
 * with the floor's top edge half a metre above its bottom); a pixel takes the
 * colour of the highest-index active shape that contains its centre (polygon:
 * not outside any face; circle: squared distance <= radius squared), white
 * otherwise; colours by role (none: grey, darker if fixated; green; blue;
 * red), alpha 255.  Joints and thrusters are not drawn. */
#define PIX 125
void k2d_ref_render(ref_sim *S, uint8_t *out) {
    const ref_config *cf = &S->cfg;
    const int P = S->P, C = S->C, N = S->N;
    const real scale = RC(0.05), x0 = RC(-3.125), y1 = RC(5.75);
    static const uint8_t role_rgb[4][3] = { { 128, 128, 128 }, { 0, 200, 0 }, { 0, 0, 220 }, { 220, 0, 0 } };
    for (int e = 0; e < cf->n_envs; ++e) {
        const int l = S->level_id[e];
        const real *pos = S->pos + (size_t)e * N * 2, *ang = S->angle + (size_t)e * N;
        real cs[32], sn[32];
        wpoly W[16];
        for (int i = 0; i < N; ++i) k2d_ref_sincos(ang[i], &cs[i], &sn[i]);
        for (int i = 0; i < P; ++i) {
            wpoly *w = &W[i];
            w->cnt = S->lv_nverts[l * P + i];
            const real *lv = S->lv_verts + ((size_t)(l * P + i) * MAX_VERTS) * 2;
            const real *ln = S->lv_normals + ((size_t)(l * P + i) * MAX_VERTS) * 2;
            for (int k = 0; k < w->cnt; ++k) {
                vec2 loc = { lv[2 * k], lv[2 * k + 1] }, nl = { ln[2 * k], ln[2 * k + 1] };
                vec2 r = rot2(cs[i], sn[i], loc);
                w->w[k].x = r.x + pos[2 * i]; w->w[k].y = r.y + pos[2 * i + 1];
                w->nrm[k] = rot2(cs[i], sn[i], nl);
                w->off[k] = dot2(w->nrm[k], w->w[k]);
            }
        }
        uint8_t *img = out + (size_t)e * PIX * PIX * 4;
        for (int r = 0; r < PIX; ++r)
            for (int c = 0; c < PIX; ++c) {
                vec2 p = { x0 + ((real)c + RC(0.5)) * scale, y1 - ((real)r + RC(0.5)) * scale };
                int hit = -1;
                for (int i = N - 1; i >= 0 && hit < 0; --i) {
                    if (!S->lv_active[l * N + i]) continue;
                    if (i < P) {
                        int inside = 1;
                        for (int k = 0; k < W[i].cnt; ++k) if (dot2(W[i].nrm[k], p) - W[i].off[k] > RC(0)) inside = 0;
                        if (inside) hit = i;
                    } else {
                        vec2 d = { p.x - pos[2 * i], p.y - pos[2 * i + 1] };
                        real rad = S->lv_radius[l * C + (i - P)];
                        if (dot2(d, d) <= rad * rad) hit = i;
                    }
                }
                uint8_t *px = img + ((size_t)r * PIX + c) * 4;
                if (hit < 0) { px[0] = px[1] = px[2] = 255; }
                else {
                    int role = S->lv_role[l * N + hit];
                    const uint8_t *rgb = role_rgb[role];
                    int dark = (role == 0 && S->lv_static[l * N + hit]);
                    px[0] = dark ? 64 : rgb[0]; px[1] = dark ? 64 : rgb[1]; px[2] = dark ? 64 : rgb[2];
                }
                px[3] = 255;
            }
    }
}

int k2d_ref_real_bytes(void) { return (int)sizeof(real); }
