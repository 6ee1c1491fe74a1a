// k2d_api.cu -- host side of the C ABI declared in include/k2d.h: validation, level build (mass
// properties, collision mask, constraint levels), buffer layout, kernel launches.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "k2d.h"
#include "k2d_kernels.cuh"

namespace k2d {

using ClassS = SizeClass<5, 2, 1, 1>;
using ClassM = SizeClass<6, 3, 2, 2>;
using ClassL = SizeClass<12, 4, 6, 2>;

constexpr int kMaxSlots = 8192;      // resident scene groups a launch may use (bounds the overflow scratch)
constexpr size_t kCtrlBytes = 4096;  // control block at the start of the state buffer: 8 x uint64 counters, the work queue words at
                                     // kQueueOffset, the counting sort's words (2 x 256 + 1) at kSortOffset
constexpr size_t kSortOffset = 1024;
constexpr size_t kQueueOffset = 128;
#ifndef K2D_CHUNK_STEPS
#define K2D_CHUNK_STEPS 8
#endif
constexpr int kChunkSteps = K2D_CHUNK_STEPS;       // steps per work item when there are more envs than resident scene groups

// run-time view of a size class
struct ClassInfo {
    int id, P, C, N, J, T, NPP, NPC, NCC, NPAIRS, NSLOTS, MASKW;
    int LV_WORDS, ST_WORDS, SCRATCH_WORDS, PTAB_WORDS;
    int LV_X, LV_IM, LV_II, LV_FR, LV_RE, LV_FLAGS, LV_DENS, LV_RAD, LV_PVX, LV_PVY, LV_PNX, LV_PNY, LV_ELEN, LV_JOINT, LV_THR, LV_MASK, LV_GB;
    int ST_JACC, ST_META, ST_WARM;
};
template <class SC>
static ClassInfo make_info(int id) {
    ClassInfo c{};
    c.id = id; c.P = SC::P; c.C = SC::C; c.N = SC::N; c.J = SC::J; c.T = SC::T;
    c.NPP = SC::NPP; c.NPC = SC::NPC; c.NCC = SC::NCC; c.NPAIRS = SC::NPAIRS; c.NSLOTS = SC::NSLOTS; c.MASKW = SC::MASKW;
    c.LV_WORDS = SC::LV_WORDS; c.ST_WORDS = SC::ST_WORDS; c.SCRATCH_WORDS = SC::SCRATCH_WORDS; c.PTAB_WORDS = SC::PTAB_WORDS;
    c.LV_X = SC::LV_X; c.LV_IM = SC::LV_IM; c.LV_II = SC::LV_II; c.LV_FR = SC::LV_FR; c.LV_RE = SC::LV_RE; c.LV_FLAGS = SC::LV_FLAGS;
    c.LV_DENS = SC::LV_DENS; c.LV_RAD = SC::LV_RAD; c.LV_PVX = SC::LV_PVX; c.LV_PVY = SC::LV_PVY; c.LV_PNX = SC::LV_PNX; c.LV_PNY = SC::LV_PNY;
    c.LV_ELEN = SC::LV_ELEN; c.LV_JOINT = SC::LV_JOINT; c.LV_THR = SC::LV_THR; c.LV_MASK = SC::LV_MASK; c.LV_GB = SC::LV_GB;
    c.ST_JACC = SC::ST_JACC; c.ST_META = SC::ST_META; c.ST_WARM = SC::ST_WARM;
    return c;
}

static bool pick_class(const k2d_config *cfg, ClassInfo *out) {
    const ClassInfo all[3] = { make_info<ClassS>(0), make_info<ClassM>(1), make_info<ClassL>(2) };
    for (const ClassInfo &c : all)
        if (cfg->n_polygons <= c.P && cfg->n_circles <= c.C && cfg->n_joints <= c.J && cfg->n_thrusters <= c.T) { *out = c; return true; }
    return false;
}

static int check_config(const k2d_config *c) {
    if (!c) return K2D_ERR_NULL;
    if (c->n_envs < 1 || c->n_polygons < 1 || c->n_polygons > K2D_MAX_POLYGONS || c->n_circles < 0 || c->n_circles > K2D_MAX_CIRCLES ||
        c->n_joints < 0 || c->n_joints > K2D_MAX_JOINTS || c->n_thrusters < 0 || c->n_thrusters > K2D_MAX_THRUSTERS ||
        c->n_actions < 1 || c->n_actions > kMaxActions || c->n_levels < 1 || c->solver_iters < 0 || c->solver_iters > 1024 ||
        (c->warm_start != 0 && c->warm_start != 1) || c->auto_reset < 0 || c->auto_reset > 2 || c->max_episode_steps < 0 ||
        c->max_fused_steps < 1 || c->frame_skip < 1 || c->device < 0 ||
        !(c->lanes_per_scene == 0 || c->lanes_per_scene == 8 || c->lanes_per_scene == 16 || c->lanes_per_scene == 32) || c->solver_batch < 0)
        return K2D_ERR_CONFIG;
    const float f[] = { c->dt, c->gravity_y, c->contact_alpha, c->contact_beta, c->slop, c->restitution_threshold, c->face_tol,
                        c->joint_alpha, c->joint_beta, c->motor_rho, c->aabb_margin, c->joint_gamma, c->dense_kappa };
    for (float v : f) if (!std::isfinite(v)) return K2D_ERR_CONFIG;
    if (!(c->dt > 0.0f) || c->aabb_margin < 0.0f || c->slop < 0.0f) return K2D_ERR_CONFIG;
    return K2D_OK;
}

// canonical pair index of shapes (a < b in canonical sense) for a scene with P polygons and C circles
static int pair_index(int P, int C, int a, int b) {
    const int npp = P * (P - 1) / 2, npc = P * C;
    if (b < P) return a * (2 * P - a - 1) / 2 + (b - a - 1);
    if (a < P) return npp + a * C + (b - P);
    const int i = a - P, j = b - P;
    return npp + npc + i * (2 * C - i - 1) / 2 + (j - i - 1);
}
static int pair_slot(int P, int C, int p) {
    const int npp = P * (P - 1) / 2;
    (void)C;
    return p < npp ? 2 * p : npp + p;
}

}  // namespace k2d

using namespace k2d;

struct k2d_state {
    k2d_config cfg;
    ClassInfo ci;
    int G, grid, groups, slots;
    unsigned wait_limit;
    size_t smem_bytes;
    cudaStream_t stream;
    unsigned char *dev_base;
    unsigned long long *dev_counters;
    unsigned int *dev_queue, *dev_chunks, *dev_sort;
    int block_threads;   // threads per block of the step kernel for this handle
    bool large_block;    // one block per SM, warps in lockstep per scheduler (enough envs to fill the device)
    int order_age;       // launches since the envs were last sorted for the work queue (0: the order is not valid)
    int *dev_ids;
    uint32_t *dev_env, *dev_scratch, *dev_levels;
    float *dev_trace;
    std::vector<uint32_t> host_levels;     // packed level records, kept for k2d_level_info and set_state
    std::vector<int> shape_map;            // config shape index -> internal shape index
    std::vector<int> pair_map;             // config pair index -> internal pair index
};

namespace k2d {

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct BufLayout { size_t ids_off, chunks_off, env_off, scratch_off, total; int slots; };
static BufLayout buffer_layout(const k2d_config *cfg, const ClassInfo &ci) {
    BufLayout b{};
    // every scene group of a launch can end up stepping an env, so the scratch covers whole blocks (up to 16 groups each)
    b.slots = ((cfg->n_envs < kMaxSlots ? cfg->n_envs : kMaxSlots) + 15) / 16 * 16;
    b.ids_off = kCtrlBytes;
    b.chunks_off = align_up(b.ids_off + (size_t)cfg->n_envs * 4, 256);
    b.env_off = align_up(b.chunks_off + (size_t)cfg->n_envs * 4, 256);
    b.scratch_off = align_up(b.env_off + (size_t)cfg->n_envs * ci.ST_WORDS * 4, 256);
    b.total = align_up(b.scratch_off + (size_t)b.slots * ci.SCRATCH_WORDS * 4, 256);
    return b;
}

static inline uint32_t f2u(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }
static inline float u2f(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

// Packs one caller level into the device record.  Mass properties: uniform lamina, evaluated in
// double in a fixed order and rounded once (area = 1/2 sum cross, I = rho/12 sum cross (a.a + a.b + b.b)).
static int pack_level(const k2d_config *cfg, const ClassInfo &ci, const k2d_level *L, uint32_t *w) {
    const int nP = cfg->n_polygons, nC = cfg->n_circles, nN = nP + nC, nJ = cfg->n_joints, nT = cfg->n_thrusters;
    std::memset(w, 0, sizeof(uint32_t) * ci.LV_WORDS);
    auto internal = [&](int i) { return i < nP ? i : ci.P + (i - nP); };
    std::vector<int> is_static(ci.N, 1), is_active(ci.N, 0);
    for (int i = 0; i < nN; ++i) {
        const int q = internal(i);
        const float pose[6] = { L->pos[i][0], L->pos[i][1], L->angle[i], L->vel[i][0], L->vel[i][1], L->angvel[i] };
        for (float v : pose) if (!std::isfinite(v)) return K2D_ERR_LEVEL;
        const bool act = L->active[i] != 0, st = L->is_static[i] != 0;
        w[ci.LV_X + 0 * ci.N + q] = f2u(pose[0]); w[ci.LV_X + 1 * ci.N + q] = f2u(pose[1]); w[ci.LV_X + 2 * ci.N + q] = f2u(pose[2]);
        // fixated shapes never move
        w[ci.LV_X + 3 * ci.N + q] = f2u(st ? 0.0f : pose[3]); w[ci.LV_X + 4 * ci.N + q] = f2u(st ? 0.0f : pose[4]);
        w[ci.LV_X + 5 * ci.N + q] = f2u(st ? 0.0f : pose[5]);
        if (!act) continue;
        if (L->role[i] < 0 || L->role[i] > 3) return K2D_ERR_LEVEL;
        const float mat[3] = { L->density[i], L->friction[i], L->restitution[i] };
        for (float v : mat) if (!std::isfinite(v) || v < 0.0f) return K2D_ERR_LEVEL;
        if (!(L->density[i] > 0.0f)) return K2D_ERR_LEVEL;
        double mass, inertia;
        uint32_t nv = 0;
        if (i < nP) {
            nv = (uint32_t)L->poly_nverts[i];
            if (nv != 3 && nv != 4) return K2D_ERR_LEVEL;
            double area2 = 0.0, second = 0.0, cxs = 0.0, cys = 0.0, ext = 0.0;
            for (uint32_t k = 0; k < nv; ++k) {
                const uint32_t k1 = (k + 1) % nv, k2 = (k + 2) % nv;
                const double x0 = L->poly_verts[i][k][0], y0 = L->poly_verts[i][k][1];
                const double x1 = L->poly_verts[i][k1][0], y1 = L->poly_verts[i][k1][1];
                const double x2 = L->poly_verts[i][k2][0], y2 = L->poly_verts[i][k2][1];
                if (!std::isfinite(x0) || !std::isfinite(y0)) return K2D_ERR_LEVEL;
                const double cr = x0 * y1 - y0 * x1;
                area2 += cr;
                second += cr * ((x0 * x0 + y0 * y0) + (x0 * x1 + y0 * y1) + (x1 * x1 + y1 * y1));
                cxs += (x0 + x1) * cr; cys += (y0 + y1) * cr;
                const double ex = x1 - x0, ey = y1 - y0;
                const double len = std::sqrt(ex * ex + ey * ey);
                if (!(len > 0.0)) return K2D_ERR_LEVEL;
                if (!((ex * (y2 - y1) - ey * (x2 - x1)) > 0.0)) return K2D_ERR_LEVEL;   // convex, counter-clockwise
                w[ci.LV_PVX + 4 * q + k] = f2u((float)x0); w[ci.LV_PVY + 4 * q + k] = f2u((float)y0);
                w[ci.LV_PNX + 4 * q + k] = f2u((float)(ey / len)); w[ci.LV_PNY + 4 * q + k] = f2u((float)(-ex / len));
                w[ci.LV_ELEN + 4 * q + k] = f2u((float)len);
                ext = std::fmax(ext, std::fmax(std::fabs(x0), std::fabs(y0)));
            }
            if (!(area2 > 0.0)) return K2D_ERR_LEVEL;
            if (std::hypot(cxs / (3.0 * area2), cys / (3.0 * area2)) > 1e-3 * ext) return K2D_ERR_LEVEL;  // centroid at the origin
            const double rho = L->density[i];
            mass = rho * (0.5 * area2);
            inertia = rho * (second / 12.0);
        } else {
            const double r = L->circle_radius[i - nP], rho = L->density[i];
            if (!std::isfinite(r) || !(r > 0.0)) return K2D_ERR_LEVEL;
            mass = rho * (3.14159265358979323846 * (r * r));
            inertia = (mass * (r * r)) * 0.5;
            w[ci.LV_RAD + (q - ci.P)] = f2u((float)r);
        }
        is_active[q] = 1; is_static[q] = st ? 1 : 0;
        w[ci.LV_IM + q] = f2u(st ? 0.0f : (float)(1.0 / mass));
        w[ci.LV_II + q] = f2u(st ? 0.0f : (float)(1.0 / inertia));
        w[ci.LV_FR + q] = f2u(L->friction[i]); w[ci.LV_RE + q] = f2u(L->restitution[i]); w[ci.LV_DENS + q] = f2u(L->density[i]);
        w[ci.LV_FLAGS + q] = F_ACTIVE | (st ? 0u : F_DYNAMIC) | ((uint32_t)L->role[i] << 2) | (nv << 4);
    }
    // the dense reward measures the distance between the first green and the first blue shape
    {
        int g = -1, b = -1;
        for (int q = ci.N - 1; q >= 0; --q) {
            if (!is_active[q]) continue;
            const uint32_t role = flag_role(w[ci.LV_FLAGS + q]);
            if (role == K2D_ROLE_GREEN) g = q;
            if (role == K2D_ROLE_BLUE) b = q;
        }
        w[ci.LV_GB] = (g >= 0 && b >= 0) ? ((uint32_t)g | ((uint32_t)b << 8) | (1u << 16)) : 0u;
    }
    // joints: "on" when both shapes exist and at least one can move; level = 1 + highest level of an earlier
    // joint sharing a movable shape (so lanes can run a level's joints at once and keep the joint order)
    std::vector<int> body_level(ci.N, 0);
    std::vector<std::pair<int, int>> joined;
    int joint_levels = 0;
    for (int j = 0; j < nJ; ++j) {
        uint32_t *jw = w + ci.LV_JOINT + kJointLevelWords * j;
        if (!L->joint_active[j]) continue;
        const int a0 = L->joint_a[j], b0 = L->joint_b[j];
        if (a0 < 0 || a0 >= nN || b0 < 0 || b0 >= nN || a0 == b0) return K2D_ERR_LEVEL;
        if (L->motor_binding[j] < 0 || L->motor_binding[j] >= cfg->n_actions) return K2D_ERR_LEVEL;
        const float v[9] = { L->joint_anchor_a[j][0], L->joint_anchor_a[j][1], L->joint_anchor_b[j][0], L->joint_anchor_b[j][1],
                             L->motor_speed[j], L->motor_power[j], L->joint_fixed_angle[j], L->joint_min[j], L->joint_max[j] };
        for (float x : v) if (!std::isfinite(x)) return K2D_ERR_LEVEL;
        if (L->joint_limited[j] && !L->joint_fixed[j] && L->joint_min[j] > L->joint_max[j]) return K2D_ERR_LEVEL;
        const int a = internal(a0), b = internal(b0);
        const bool on = is_active[a] && is_active[b] && !(is_static[a] && is_static[b]);
        int lvl = 0;
        if (on) {
            lvl = 1;
            if (!is_static[a]) lvl = std::max(lvl, body_level[a] + 1);
            if (!is_static[b]) lvl = std::max(lvl, body_level[b] + 1);
            if (!is_static[a]) body_level[a] = lvl;
            if (!is_static[b]) body_level[b] = lvl;
            joint_levels = std::max(joint_levels, lvl);
        }
        jw[0] = (uint32_t)a | ((uint32_t)b << 8) | ((uint32_t)L->motor_binding[j] << 16) | ((on ? 1u : 0u) << 24) | ((uint32_t)lvl << 25) | (1u << 28) |
                ((is_static[a] ? 0u : 1u) << 29) | ((is_static[b] ? 0u : 1u) << 30) |
                (((L->joint_fixed[j] || L->joint_limited[j]) ? 1u : 0u) << 31);
        for (int k = 0; k < 9; ++k) jw[1 + k] = f2u(v[k]);
        jw[10] = L->joint_fixed[j] ? 1u : (L->joint_limited[j] ? 2u : 0u);
        joined.emplace_back(a, b);
    }
    w[ci.LV_GB] |= (uint32_t)std::min(joint_levels, 7) << 24;      // what the launch's env order sorts by (with the touching pairs)
    std::fill(body_level.begin(), body_level.end(), 0);
    for (int t = 0; t < nT; ++t) {
        uint32_t *tw = w + ci.LV_THR + 8 * t;
        if (!L->thr_active[t]) continue;
        const int s0 = L->thr_shape[t];
        if (s0 < 0 || s0 >= nN) return K2D_ERR_LEVEL;
        if (L->thr_binding[t] < 0 || L->thr_binding[t] >= cfg->n_actions) return K2D_ERR_LEVEL;
        const float v[4] = { L->thr_pos[t][0], L->thr_pos[t][1], L->thr_rot[t], L->thr_power[t] };
        for (float x : v) if (!std::isfinite(x)) return K2D_ERR_LEVEL;
        const int q = internal(s0);
        const bool on = is_active[q] != 0;
        int lvl = 0;
        if (on) { lvl = body_level[q] + 1; body_level[q] = lvl; }
        const double phi = L->thr_rot[t];
        tw[0] = (uint32_t)q | ((uint32_t)L->thr_binding[t] << 8) | ((on ? 1u : 0u) << 16) | ((uint32_t)lvl << 17) | (1u << 20);
        tw[1] = f2u(v[0]); tw[2] = f2u(v[1]); tw[3] = f2u((float)std::cos(phi)); tw[4] = f2u((float)std::sin(phi)); tw[5] = f2u(v[3]);
    }
    // which pairs may collide: both shapes present, not both fixated, not joined (paper: joined shapes do not collide)
    for (int a = 0; a < ci.N; ++a)
        for (int b = a + 1; b < ci.N; ++b) {
            if (!is_active[a] || !is_active[b] || (is_static[a] && is_static[b])) continue;
            bool jn = false;
            for (auto &pr : joined) jn = jn || (pr.first == a && pr.second == b) || (pr.first == b && pr.second == a);
            if (jn) continue;
            const int p = pair_index(ci.P, ci.C, a, b);
            w[ci.LV_MASK + (p >> 5)] |= 1u << (p & 31);
        }
    return K2D_OK;
}

template <class SC, int G>
static cudaError_t launch_step(const k2d_state *s, const StepParams &prm) {
    constexpr int LARGE = step_block_threads<SC, G>();
    if (s->large_block) k2d_step_kernel<SC, G, LARGE><<<s->grid, LARGE, s->smem_bytes, s->stream>>>(prm);
    else k2d_step_kernel<SC, G, kSmallBlock><<<s->grid, kSmallBlock, s->smem_bytes, s->stream>>>(prm);
    return cudaGetLastError();
}
// Launch shape of the step kernel for this handle.  With enough envs to give every scene group of the device one, the kernel
// runs as one block per SM whose warps step in lockstep per scheduler; with fewer, as small blocks spread over all SMs.
template <class SC, int G>
static cudaError_t setup_step(k2d_state *s, int num_sms) {
    constexpr int LARGE = step_block_threads<SC, G>();
    s->large_block = LARGE > kSmallBlock && s->cfg.n_envs >= num_sms * (LARGE / G) && s->slots >= num_sms * (LARGE / G);
    const int threads = s->large_block ? LARGE : kSmallBlock, GPB = threads / G;
    s->block_threads = threads;
    s->smem_bytes = step_block_smem<SC, G>(threads);
    cudaError_t err;
    int per_sm = 0;
    if (s->large_block) {
        err = cudaFuncSetAttribute(k2d_step_kernel<SC, G, LARGE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s->smem_bytes);
        if (err != cudaSuccess) return err;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k2d_step_kernel<SC, G, LARGE>, threads, s->smem_bytes);
    } else {
        err = cudaFuncSetAttribute(k2d_step_kernel<SC, G, kSmallBlock>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s->smem_bytes);
        if (err != cudaSuccess) return err;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k2d_step_kernel<SC, G, kSmallBlock>, threads, s->smem_bytes);
    }
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    int grid = num_sms * per_sm;
    const int need = (s->cfg.n_envs + GPB - 1) / GPB;
    if (grid > need) grid = need;
    if (grid * GPB > s->slots) grid = s->slots / GPB;
    if (grid < 1) grid = 1;
    s->grid = grid;
    s->groups = grid * GPB;
    return cudaSuccess;
}

template <class SC>
static cudaError_t launch_obs(const k2d_state *s, float *dev_obs) {
    const k2d_config &c = s->cfg;
    const int epb = kObsEnvsPerBlock, grid = (c.n_envs + epb - 1) / epb;
    const int width = (c.n_polygons + c.n_circles) * 29 + c.n_joints * 2 * (11 + c.n_actions) + c.n_thrusters * 6;
    const size_t smem = sizeof(float) * epb * obs_image_stride(width, SC::N);
    k2d_obs_kernel<SC><<<grid, kObsThreads, smem, s->stream>>>(s->dev_env, s->dev_levels, dev_obs, c.n_envs, c.n_actions, c.n_polygons,
                                                              c.n_circles, c.n_joints, c.n_thrusters);
    return cudaGetLastError();
}

template <class SC>
static cudaError_t launch_render(const k2d_state *s, uint32_t *out) {
    k2d_render_kernel<SC><<<s->cfg.n_envs, kRenderThreads, 0, s->stream>>>(s->dev_env, s->dev_levels, out, s->cfg.n_envs);
    return cudaGetLastError();
}

// Kernel arguments of one k2d_step launch.  With more envs than resident scene groups the launch is cut
// into chunks of kChunkSteps steps, so that the groups can balance the work between them.
static StepParams step_params(const k2d_state *s, const float *dev_actions, int n_steps, float *dev_reward, uint8_t *dev_done,
                              uint32_t *scratch, int discrete = 0) {
    const k2d_config &c = s->cfg;
    StepParams prm{};
    prm.state = s->dev_env; prm.levels = s->dev_levels; prm.actions = dev_actions; prm.reward = dev_reward; prm.done = dev_done;
    prm.counters = s->dev_counters; prm.queue = s->dev_queue; prm.chunks_done = s->dev_chunks; prm.scratch = scratch; prm.trace = s->dev_trace;
    prm.n_envs = c.n_envs; prm.n_steps = n_steps; prm.n_actions = c.n_actions; prm.n_levels = c.n_levels;
    prm.obs = nullptr; prm.n_polygons = c.n_polygons; prm.n_circles = c.n_circles; prm.n_joints = c.n_joints; prm.n_thrusters = c.n_thrusters;
    prm.discrete = discrete; prm.dense_kappa = c.dense_kappa; prm.frame_skip = c.frame_skip;
    prm.order = nullptr;
    prm.chunk_steps = n_steps; prm.n_chunks = 1; prm.wait_limit = s->wait_limit; prm.n_slots = scratch == s->dev_scratch ? s->slots : K2D_STATIC_SCRATCH_MAX_ENVS;
    {
        const int n_slots = c.n_polygons * (c.n_polygons - 1) + c.n_polygons * c.n_circles + c.n_circles * (c.n_circles - 1) / 2;
        prm.n_batches = c.solver_batch > 0 ? (n_slots + c.solver_batch - 1) / c.solver_batch : 0;
        if (c.solver_batch > 0 && prm.n_batches < 1) prm.n_batches = 1;
    }
    if (c.n_envs > s->groups && n_steps > kChunkSteps) {
        const int n_chunks = (n_steps + kChunkSteps - 1) / kChunkSteps;
        if ((unsigned long long)c.n_envs * (unsigned long long)n_chunks + (unsigned long long)s->groups < 0xffffffffULL) {
            prm.chunk_steps = kChunkSteps; prm.n_chunks = n_chunks;
        }
    }
    prm.solver_iters = c.solver_iters; prm.warm_start = c.warm_start; prm.auto_reset = c.auto_reset; prm.max_episode_steps = c.max_episode_steps;
    prm.dt = c.dt; prm.gdt = c.gravity_y * c.dt; prm.contact_alpha = c.contact_alpha; prm.contact_beta = c.contact_beta; prm.slop = c.slop;
    prm.rest_thr = c.restitution_threshold; prm.face_tol = c.face_tol; prm.joint_alpha = c.joint_alpha; prm.joint_beta = c.joint_beta; prm.joint_gamma = c.joint_gamma;
    prm.motor_rho = c.motor_rho; prm.aabb_margin = c.aabb_margin; prm.seed = c.seed; prm.env_offset = c.env_offset;
    return prm;
}

// Launches of at least kOrderMinSteps steps with two or more scenes per warp and more envs than the device holds scene groups
// first sort the envs by what their steps cost (see k2d_order_count_kernel); the order lives in the words that k2d_reset uses
// for the level ids, free between resets.
constexpr int kOrderMinSteps = 8, kOrderShortLaunches = 16;
template <class SC>
static cudaError_t launch_order(const k2d_state *s) {
    const int n = s->cfg.n_envs, grid = (n + kOrderThreads - 1) / kOrderThreads;
    k2d_order_count_kernel<SC><<<grid, kOrderThreads, 0, s->stream>>>(s->dev_env, s->dev_levels, s->dev_sort, n, s->cfg.n_levels);
    k2d_order_place_kernel<SC><<<grid, kOrderThreads, 0, s->stream>>>(s->dev_env, s->dev_levels, s->dev_sort, s->dev_ids, n, s->cfg.n_levels);
    return cudaGetLastError();
}
// with one scene per warp and small blocks nothing runs in lockstep, and with no more envs than groups every group gets one env anyway
static bool uses_order(const k2d_state *s) {
    // one block per SM: from one and a half waves of envs on (measured on L scenes, sorted against unsorted env-steps/s:
    // 7400 envs 114.6 M / 123.6 M, 8192 132.1 M / 135.8 M, 9000 140.3 M / 137.6 M, 12000 152.9 M / 141.9 M, 16384 158.3 M / 146.8 M)
    if (s->large_block) return 2 * (long long)s->cfg.n_envs > 3 * (long long)s->groups;
    return s->G < 32 && s->cfg.n_envs > s->groups;
}
// a short launch reuses the order of an earlier one (what an env's step costs changes slowly) and sorts again every
// kOrderShortLaunches launches; k2d_reset, which uses the same words, makes the next launch sort
static bool reuses_order(const k2d_state *s, int n_steps) {
    return n_steps < kOrderMinSteps && s->order_age > 0 && s->order_age < kOrderShortLaunches;
}
static cudaError_t order_envs(k2d_state *s, StepParams &prm) {
    if (!uses_order(s)) return cudaSuccess;
    prm.order = s->dev_ids;
    if (reuses_order(s, prm.n_steps)) { ++s->order_age; return cudaSuccess; }
    s->order_age = 1;
    return s->ci.id == 0 ? launch_order<ClassS>(s) : s->ci.id == 1 ? launch_order<ClassM>(s) : launch_order<ClassL>(s);
}

#define K2D_DISPATCH(FN, s, ...)                                                                      \
    ((s)->ci.id == 0 ? ((s)->G == 32 ? FN<ClassS, 32>(__VA_ARGS__) : (s)->G == 16 ? FN<ClassS, 16>(__VA_ARGS__) : FN<ClassS, 8>(__VA_ARGS__)) \
   : (s)->ci.id == 1 ? ((s)->G == 32 ? FN<ClassM, 32>(__VA_ARGS__) : (s)->G == 16 ? FN<ClassM, 16>(__VA_ARGS__) : FN<ClassM, 8>(__VA_ARGS__)) \
                     : ((s)->G == 32 ? FN<ClassL, 32>(__VA_ARGS__) : (s)->G == 16 ? FN<ClassL, 16>(__VA_ARGS__) : FN<ClassL, 8>(__VA_ARGS__)))

// does the observation image of the handle's scenes fit into the part of a scene's shared-memory region the step kernel can spare for it?
template <class SC, int G>
static bool obs_fits(const k2d_state *s) {
    return SC::WVX + k2d_obs_floats(&s->cfg) <= region_words<SC, G>();
}

}  // namespace k2d

#define CUDA_OK(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { std::fprintf(stderr, "k2d: %s failed: %s\n", #call, cudaGetErrorString(e_)); return K2D_ERR_CUDA; } } while (0)

extern "C" {

int k2d_default_config(k2d_config *cfg, int32_t n_envs, int32_t n_polygons, int32_t n_circles, int32_t n_joints, int32_t n_thrusters) {
    if (!cfg) return K2D_ERR_NULL;
    std::memset(cfg, 0, sizeof(*cfg));
    cfg->n_envs = n_envs; cfg->n_polygons = n_polygons; cfg->n_circles = n_circles; cfg->n_joints = n_joints; cfg->n_thrusters = n_thrusters;
    cfg->n_actions = n_joints + n_thrusters > 0 ? n_joints + n_thrusters : 1;
    cfg->n_levels = n_envs;
    cfg->solver_iters = 8; cfg->warm_start = 1; cfg->auto_reset = K2D_RESET_NONE; cfg->max_episode_steps = 0; cfg->max_fused_steps = 64; cfg->frame_skip = 1;
    cfg->dt = 1.0f / 60.0f; cfg->gravity_y = -9.81f;
    cfg->contact_alpha = 6.0f; cfg->contact_beta = 0.1f; cfg->slop = 0.005f; cfg->restitution_threshold = 1.0f; cfg->face_tol = 1e-3f;
    cfg->joint_alpha = 6.0f; cfg->joint_beta = 0.1f; cfg->joint_gamma = 6.0f; cfg->motor_rho = 1.0f; cfg->aabb_margin = 0.01f;
    return check_config(cfg);
}

size_t k2d_state_bytes(const k2d_config *cfg) {
    ClassInfo ci;
    if (check_config(cfg) != K2D_OK || !pick_class(cfg, &ci)) return 0;
    return buffer_layout(cfg, ci).total;
}

size_t k2d_state_bytes_no_scratch(const k2d_config *cfg) {
    ClassInfo ci;
    if (check_config(cfg) != K2D_OK || !pick_class(cfg, &ci)) return 0;
    return buffer_layout(cfg, ci).scratch_off;
}

size_t k2d_level_pool_bytes(const k2d_config *cfg) {
    ClassInfo ci;
    if (check_config(cfg) != K2D_OK || !pick_class(cfg, &ci)) return 0;
    return align_up((size_t)cfg->n_levels * ci.LV_WORDS * 4, 256);
}

int k2d_obs_floats(const k2d_config *cfg) {
    if (check_config(cfg) != K2D_OK) return 0;
    return (cfg->n_polygons + cfg->n_circles) * 29 + cfg->n_joints * 2 * (11 + cfg->n_actions) + cfg->n_thrusters * 6;
}

int k2d_canonical_words(const k2d_config *cfg) {
    if (check_config(cfg) != K2D_OK) return 0;
    const int P = cfg->n_polygons, C = cfg->n_circles, N = P + C;
    const int slots = P * (P - 1) + P * C + C * (C - 1) / 2;
    return 6 * N + 2 * slots + 3 * cfg->n_joints + 4;
}

int k2d_create(const k2d_config *cfg, void *dev_state_buf, void *dev_level_pool_buf, const k2d_level *host_levels, k2d_state **out) {
    if (!cfg || !dev_state_buf || !dev_level_pool_buf || !host_levels || !out) return K2D_ERR_NULL;
    *out = nullptr;
    int rc = check_config(cfg);
    if (rc != K2D_OK) return rc;
    ClassInfo ci;
    if (!pick_class(cfg, &ci)) return K2D_ERR_CONFIG;
    if (((uintptr_t)dev_state_buf & 15) || ((uintptr_t)dev_level_pool_buf & 15)) return K2D_ERR_ALIGN;
    k2d_state *s = new (std::nothrow) k2d_state();
    if (!s) return K2D_ERR_ARG;
    s->cfg = *cfg; s->ci = ci;
    s->G = cfg->lanes_per_scene ? cfg->lanes_per_scene : 16;
    s->stream = (cudaStream_t)cfg->cuda_stream;
    s->wait_limit = kWaitLimit;
    s->dev_trace = nullptr;
    // index maps between the caller's scene dimensions and the internal size class
    const int nP = cfg->n_polygons, nC = cfg->n_circles, nN = nP + nC;
    s->shape_map.resize(nN);
    for (int i = 0; i < nN; ++i) s->shape_map[i] = i < nP ? i : ci.P + (i - nP);
    s->pair_map.resize(nN * (nN - 1) / 2);
    for (int a = 0; a < nN; ++a)
        for (int b = a + 1; b < nN; ++b)
            s->pair_map[pair_index(nP, nC, a, b)] = pair_index(ci.P, ci.C, s->shape_map[a], s->shape_map[b]);
    s->host_levels.assign((size_t)cfg->n_levels * ci.LV_WORDS, 0u);
    for (int l = 0; l < cfg->n_levels; ++l) {
        rc = pack_level(cfg, ci, host_levels + l, s->host_levels.data() + (size_t)l * ci.LV_WORDS);
        if (rc != K2D_OK) { delete s; return rc; }
    }
    const BufLayout bl = buffer_layout(cfg, ci);
    s->slots = bl.slots;
    s->dev_base = (unsigned char *)dev_state_buf;
    s->dev_counters = (unsigned long long *)s->dev_base;
    s->dev_queue = (unsigned int *)(s->dev_base + kQueueOffset);
    s->dev_sort = (unsigned int *)(s->dev_base + kSortOffset);
    s->dev_chunks = (unsigned int *)(s->dev_base + bl.chunks_off);
    s->dev_ids = (int *)(s->dev_base + bl.ids_off);
    s->dev_env = (uint32_t *)(s->dev_base + bl.env_off);
    s->dev_scratch = (uint32_t *)(s->dev_base + bl.scratch_off);
    s->dev_levels = (uint32_t *)dev_level_pool_buf;
    cudaError_t err = cudaSetDevice(cfg->device);
    int num_sms = 0;
    if (err == cudaSuccess) err = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, cfg->device);
    // default lanes per scene: a warp per scene while the device has warps to spare (measured on B200: faster below
    // about 48 envs per SM for the largest size class, 24 for the smaller ones), two scenes per warp beyond
    // default lanes per scene: two scenes per warp once they fill the device's one-block-per-SM form (40 scenes per SM) with
    // some to spare, one scene per warp below that (measured, env-steps/s with 16 against 32 lanes: L x 8192 132.8 M / 107.2 M,
    // L x 6144 99.1 M / 103.3 M, L x 4096 70.3 M / 97.9 M, M x 4096 112.8 M / 143.3 M, S x 4096 147.7 M / 164.9 M)
    if (err == cudaSuccess && !cfg->lanes_per_scene) s->G = (cfg->n_envs < (kLargeBlock / 16) * num_sms * 9 / 8) ? 32 : 16;
    if (err == cudaSuccess) err = K2D_DISPATCH(setup_step, s, s, num_sms);
    if (err == cudaSuccess) err = cudaMemcpyAsync(s->dev_levels, s->host_levels.data(), s->host_levels.size() * 4, cudaMemcpyHostToDevice, s->stream);
    if (err == cudaSuccess) err = cudaStreamSynchronize(s->stream);
    if (err != cudaSuccess) { std::fprintf(stderr, "k2d_create: %s\n", cudaGetErrorString(err)); delete s; return K2D_ERR_CUDA; }
    rc = k2d_reset(s, nullptr);
    if (rc != K2D_OK) { delete s; return rc; }
    *out = s;
    return K2D_OK;
}

int k2d_reset(k2d_state *s, const int32_t *host_level_ids) {
    if (!s) return K2D_ERR_NULL;
    const int E = s->cfg.n_envs;
    if (host_level_ids)
        for (int e = 0; e < E; ++e) if (host_level_ids[e] < 0 || host_level_ids[e] >= s->cfg.n_levels) return K2D_ERR_ARG;
    CUDA_OK(cudaSetDevice(s->cfg.device));
    CUDA_OK(cudaMemsetAsync(s->dev_base, 0, kCtrlBytes, s->stream));
    s->order_age = 0;
#ifdef K2D_CHECKED
    { const unsigned int zero = 0u; CUDA_OK(cudaMemcpyToSymbolAsync(k2d_check_bits, &zero, sizeof(zero), 0, cudaMemcpyHostToDevice, s->stream)); }
#endif
    CUDA_OK(cudaMemsetAsync(s->dev_chunks, 0, (size_t)E * 4, s->stream));
    if (host_level_ids) CUDA_OK(cudaMemcpyAsync(s->dev_ids, host_level_ids, (size_t)E * 4, cudaMemcpyHostToDevice, s->stream));
    const int *ids = host_level_ids ? s->dev_ids : nullptr;
    if (s->ci.id == 0) k2d_reset_kernel<ClassS><<<E, 64, 0, s->stream>>>(s->dev_env, s->dev_levels, ids, E, s->cfg.n_levels);
    else if (s->ci.id == 1) k2d_reset_kernel<ClassM><<<E, 64, 0, s->stream>>>(s->dev_env, s->dev_levels, ids, E, s->cfg.n_levels);
    else k2d_reset_kernel<ClassL><<<E, 64, 0, s->stream>>>(s->dev_env, s->dev_levels, ids, E, s->cfg.n_levels);
    CUDA_OK(cudaGetLastError());
    CUDA_OK(cudaStreamSynchronize(s->stream));
    return K2D_OK;
}

int k2d_step(k2d_state *s, const float *dev_actions, int32_t n_steps, float *dev_reward, uint8_t *dev_done) {
    if (!s || !dev_actions || !dev_reward || !dev_done) return K2D_ERR_NULL;
    if (n_steps < 1 || n_steps > s->cfg.max_fused_steps) return K2D_ERR_STEPS;
    if (((uintptr_t)dev_actions & 3) || ((uintptr_t)dev_reward & 3)) return K2D_ERR_ALIGN;
    CUDA_OK(cudaSetDevice(s->cfg.device));
    StepParams prm = step_params(s, dev_actions, n_steps, dev_reward, dev_done, s->dev_scratch);
    CUDA_OK(order_envs(s, prm));
    CUDA_OK(K2D_DISPATCH(launch_step, s, s, prm));
    return K2D_OK;
}

int k2d_step_obs(k2d_state *s, const float *dev_actions, int32_t n_steps, float *dev_reward, uint8_t *dev_done, float *dev_obs) {
    if (!s || !dev_actions || !dev_reward || !dev_done || !dev_obs) return K2D_ERR_NULL;
    if (n_steps < 1 || n_steps > s->cfg.max_fused_steps) return K2D_ERR_STEPS;
    if (((uintptr_t)dev_actions & 3) || ((uintptr_t)dev_reward & 3) || ((uintptr_t)dev_obs & 3)) return K2D_ERR_ALIGN;
    CUDA_OK(cudaSetDevice(s->cfg.device));
    StepParams prm = step_params(s, dev_actions, n_steps, dev_reward, dev_done, s->dev_scratch);
    const bool fused = K2D_DISPATCH(obs_fits, s, s);
    if (fused) prm.obs = dev_obs;
    CUDA_OK(order_envs(s, prm));
    CUDA_OK(K2D_DISPATCH(launch_step, s, s, prm));
    if (!fused) return k2d_obs(s, dev_obs);       // scenes whose observation is wider than the region's spare part: a second launch
    return K2D_OK;
}

int k2d_obs(k2d_state *s, float *dev_obs) {
    if (!s || !dev_obs) return K2D_ERR_NULL;
    if ((uintptr_t)dev_obs & 3) return K2D_ERR_ALIGN;
    CUDA_OK(cudaSetDevice(s->cfg.device));
    CUDA_OK(s->ci.id == 0 ? launch_obs<ClassS>(s, dev_obs) : s->ci.id == 1 ? launch_obs<ClassM>(s, dev_obs) : launch_obs<ClassL>(s, dev_obs));
    return K2D_OK;
}

int k2d_render(k2d_state *s, uint8_t *dev_pixels) {
    if (!s || !dev_pixels) return K2D_ERR_NULL;
    if ((uintptr_t)dev_pixels & 3) return K2D_ERR_ALIGN;
    CUDA_OK(cudaSetDevice(s->cfg.device));
    const int E = s->cfg.n_envs;
    uint32_t *out = reinterpret_cast<uint32_t *>(dev_pixels);
    CUDA_OK(s->ci.id == 0 ? launch_render<ClassS>(s, out) : s->ci.id == 1 ? launch_render<ClassM>(s, out) : launch_render<ClassL>(s, out));
    return K2D_OK;
}

int k2d_get_state(k2d_state *s, void *host_canonical) {
    if (!s || !host_canonical) return K2D_ERR_NULL;
    const k2d_config &c = s->cfg; const ClassInfo &ci = s->ci;
    const int nP = c.n_polygons, nC = c.n_circles, nN = nP + nC, nJ = c.n_joints;
    const int n_slots = nP * (nP - 1) + nP * nC + nC * (nC - 1) / 2, n_pairs = nN * (nN - 1) / 2;
    const int cw = k2d_canonical_words(&c);
    std::vector<uint32_t> raw((size_t)c.n_envs * ci.ST_WORDS);
    CUDA_OK(cudaSetDevice(c.device));
    CUDA_OK(cudaStreamSynchronize(s->stream));
    CUDA_OK(cudaMemcpy(raw.data(), s->dev_env, raw.size() * 4, cudaMemcpyDeviceToHost));
    std::vector<int> inv_pair(ci.NPAIRS, -1);
    for (int p = 0; p < n_pairs; ++p) inv_pair[s->pair_map[p]] = p;
    uint32_t *outw = (uint32_t *)host_canonical;
    for (int e = 0; e < c.n_envs; ++e) {
        const uint32_t *st = raw.data() + (size_t)e * ci.ST_WORDS;
        uint32_t *o = outw + (size_t)e * cw;
        std::memset(o, 0, sizeof(uint32_t) * cw);
        for (int i = 0; i < nN; ++i) {
            const int q = s->shape_map[i];
            o[2 * i] = st[0 * ci.N + q]; o[2 * i + 1] = st[1 * ci.N + q];
            o[2 * nN + i] = st[2 * ci.N + q];
            o[3 * nN + 2 * i] = st[3 * ci.N + q]; o[3 * nN + 2 * i + 1] = st[4 * ci.N + q];
            o[5 * nN + i] = st[5 * ci.N + q];
        }
        uint32_t *acc = o + 6 * nN;
        const int nwarm = (int)st[ci.ST_META + 4];
        for (int k = 0; k < nwarm && k < ci.NPAIRS; ++k) {
            const uint32_t *wr = st + ci.ST_WARM + kWarmWords * k;
            const int p = (wr[0] < (uint32_t)ci.NPAIRS) ? inv_pair[wr[0]] : -1;
            if (p < 0) continue;
            const int slot = pair_slot(nP, nC, p);
            acc[2 * slot] = wr[1]; acc[2 * slot + 1] = wr[2];
            if (p < nP * (nP - 1) / 2) { acc[2 * slot + 2] = wr[3]; acc[2 * slot + 3] = wr[4]; }
        }
        uint32_t *jacc = acc + 2 * n_slots;
        for (int j = 0; j < 3 * nJ; ++j) jacc[j] = st[ci.ST_JACC + j];
        uint32_t *meta = jacc + 3 * nJ;
        for (int k = 0; k < 4; ++k) meta[k] = st[ci.ST_META + k];
    }
    return K2D_OK;
}

int k2d_set_state(k2d_state *s, const void *host_canonical) {
    if (!s || !host_canonical) return K2D_ERR_NULL;
    const k2d_config &c = s->cfg; const ClassInfo &ci = s->ci;
    const int nP = c.n_polygons, nC = c.n_circles, nN = nP + nC, nJ = c.n_joints;
    const int n_slots = nP * (nP - 1) + nP * nC + nC * (nC - 1) / 2, n_pairs = nN * (nN - 1) / 2;
    const int cw = k2d_canonical_words(&c);
    const uint32_t *inw = (const uint32_t *)host_canonical;
    for (int e = 0; e < c.n_envs; ++e) {
        const int lvl = (int)inw[(size_t)e * cw + cw - 2];
        if (lvl < 0 || lvl >= c.n_levels) return K2D_ERR_ARG;
    }
    std::vector<uint32_t> raw((size_t)c.n_envs * ci.ST_WORDS, 0u);
    for (int e = 0; e < c.n_envs; ++e) {
        uint32_t *st = raw.data() + (size_t)e * ci.ST_WORDS;
        const uint32_t *o = inw + (size_t)e * cw;
        const int lvl = (int)o[cw - 2];
        // shapes outside the caller's dimensions keep their level pose
        const uint32_t *lv = s->host_levels.data() + (size_t)lvl * ci.LV_WORDS;
        for (int i = 0; i < 6 * ci.N; ++i) st[i] = lv[ci.LV_X + i];
        for (int i = 0; i < nN; ++i) {
            const int q = s->shape_map[i];
            st[0 * ci.N + q] = o[2 * i]; st[1 * ci.N + q] = o[2 * i + 1];
            st[2 * ci.N + q] = o[2 * nN + i];
            st[3 * ci.N + q] = o[3 * nN + 2 * i]; st[4 * ci.N + q] = o[3 * nN + 2 * i + 1];
            st[5 * ci.N + q] = o[5 * nN + i];
        }
        const uint32_t *acc = o + 6 * nN;
        int nwarm = 0;
        for (int p = 0; p < n_pairs; ++p) {      // config pair order maps monotonically to internal pair order
            const int slot = pair_slot(nP, nC, p);
            const bool two = p < nP * (nP - 1) / 2;
            const uint32_t v[4] = { acc[2 * slot], acc[2 * slot + 1], two ? acc[2 * slot + 2] : 0u, two ? acc[2 * slot + 3] : 0u };
            if (!((v[0] | v[1] | v[2] | v[3]) & 0x7fffffffu)) continue;
            uint32_t *wr = st + ci.ST_WARM + kWarmWords * nwarm++;
            wr[0] = (uint32_t)s->pair_map[p]; wr[1] = v[0]; wr[2] = v[1]; wr[3] = v[2]; wr[4] = v[3];
        }
        const uint32_t *jacc = acc + 2 * n_slots;
        for (int j = 0; j < 3 * nJ; ++j) st[ci.ST_JACC + j] = jacc[j];
        const uint32_t *meta = jacc + 3 * nJ;
        for (int k = 0; k < 4; ++k) st[ci.ST_META + k] = meta[k];
        st[ci.ST_META + 4] = (uint32_t)nwarm;
    }
    CUDA_OK(cudaSetDevice(c.device));
    CUDA_OK(cudaStreamSynchronize(s->stream));
    CUDA_OK(cudaMemcpy(s->dev_env, raw.data(), raw.size() * 4, cudaMemcpyHostToDevice));
    return K2D_OK;
}

int k2d_status(k2d_state *s, int64_t *host_counts) {
    if (!s || !host_counts) return K2D_ERR_NULL;
    CUDA_OK(cudaSetDevice(s->cfg.device));
    CUDA_OK(cudaStreamSynchronize(s->stream));
    CUDA_OK(cudaMemcpy(host_counts, s->dev_counters, 8 * sizeof(int64_t), cudaMemcpyDeviceToHost));
    unsigned int queue[4] = { 0u, 0u, 0u, 0u };
    CUDA_OK(cudaMemcpy(queue, s->dev_queue, sizeof(queue), cudaMemcpyDeviceToHost));
#ifdef K2D_CHECKED
    unsigned int bits = 0u;
    CUDA_OK(cudaMemcpyFromSymbol(&bits, k2d_check_bits, sizeof(bits)));
    if (bits) { std::fprintf(stderr, "k2d_status: index checks failed, bits 0x%x\n", bits); return K2D_ERR_CHECK; }
#endif
    return queue[Q_ERROR] ? K2D_ERR_WAIT : K2D_OK;
}

int k2d_level_info(const k2d_config *cfg, const k2d_level *host_level, float *host_inv_mass, float *host_inv_inertia, uint8_t *host_collide) {
    if (!cfg || !host_level) return K2D_ERR_NULL;
    int rc = check_config(cfg);
    if (rc != K2D_OK) return rc;
    ClassInfo ci;
    if (!pick_class(cfg, &ci)) return K2D_ERR_CONFIG;
    std::vector<uint32_t> rec(ci.LV_WORDS);
    rc = pack_level(cfg, ci, host_level, rec.data());
    if (rc != K2D_OK) return rc;
    const uint32_t *lv = rec.data();
    const int nP = cfg->n_polygons, nC = cfg->n_circles, nN = nP + nC;
    auto internal = [&](int i) { return i < nP ? i : ci.P + (i - nP); };
    for (int i = 0; i < nN; ++i) {
        if (host_inv_mass) host_inv_mass[i] = u2f(lv[ci.LV_IM + internal(i)]);
        if (host_inv_inertia) host_inv_inertia[i] = u2f(lv[ci.LV_II + internal(i)]);
    }
    if (host_collide)
        for (int a = 0; a < nN; ++a)
            for (int b = a + 1; b < nN; ++b) {
                const int q = pair_index(ci.P, ci.C, internal(a), internal(b));
                host_collide[pair_index(nP, nC, a, b)] = (uint8_t)((lv[ci.LV_MASK + (q >> 5)] >> (q & 31)) & 1u);
            }
    return K2D_OK;
}

int k2d_set_trace(k2d_state *s, float *dev_trace) {
    if (!s) return K2D_ERR_NULL;
    s->dev_trace = dev_trace;
    return K2D_OK;
}

int k2d_trace_slots(const k2d_state *s) { return s ? s->ci.NSLOTS : 0; }

int k2d_is_checked_build(void) {
#ifdef K2D_CHECKED
    return 1;
#else
    return 0;
#endif
}

int k2d_resident_groups(const k2d_state *s) { return s ? s->groups : 0; }
int k2d_lanes_per_scene(const k2d_state *s) { return s ? s->G : 0; }
int k2d_items_per_ticket(const k2d_state *s) { return s ? (s->block_threads / 128) * (32 / s->G) : 0; }
int k2d_step_launches(const k2d_state *s, int32_t n_steps) {
    if (!s) return 0;
    return (uses_order(s) && !reuses_order(s, n_steps)) ? 3 : 1;
}

int k2d_phase_cycles(k2d_state *s, uint64_t *host_cycles, int32_t n) {
    if (!s || !host_cycles) return K2D_ERR_NULL;
    if (n < 0 || n > K2D_PHASES) return K2D_ERR_ARG;
    static_assert(K2D_PHASES == PH_COUNT, "the header's phase count is the kernels'");
#ifdef K2D_PHASE_CLOCKS
    CUDA_OK(cudaSetDevice(s->cfg.device));
    CUDA_OK(cudaStreamSynchronize(s->stream));
    unsigned long long sums[PH_COUNT];
    CUDA_OK(cudaMemcpyFromSymbol(sums, k2d_phase_sums, sizeof(sums)));
    for (int i = 0; i < n; ++i) host_cycles[i] = (uint64_t)sums[i];
    std::memset(sums, 0, sizeof(sums));
    CUDA_OK(cudaMemcpyToSymbol(k2d_phase_sums, sums, sizeof(sums)));
    return K2D_OK;
#else
    for (int i = 0; i < n; ++i) host_cycles[i] = 0;
    return K2D_ERR_BUILD;
#endif
}

int k2d_set_wait_limit(k2d_state *s, uint32_t polls) {
    if (!s) return K2D_ERR_NULL;
    s->wait_limit = polls < 64u ? 64u : polls;
    return K2D_OK;
}

int k2d_eval_sincos_tanh(const float *dev_x, int32_t n, float *dev_cos, float *dev_sin, float *dev_tanh, void *cuda_stream) {
    if (!dev_x) return K2D_ERR_NULL;
    if (n < 1) return K2D_ERR_ARG;
    k2d_eval_kernel<<<(n + 255) / 256, 256, 0, (cudaStream_t)cuda_stream>>>(dev_x, n, dev_cos, dev_sin, dev_tanh);
    CUDA_OK(cudaGetLastError());
    return K2D_OK;
}

// ---- k2d_step for callers that cannot provide the overflow scratch: it lives in the library image.
// One array per device that loads the library, held until the process exits.
static __device__ __align__(256) uint32_t k2d_static_scratch[(size_t)K2D_STATIC_SCRATCH_MAX_ENVS * ClassL::SCRATCH_WORDS];
static std::mutex k2d_static_mutex;
static uint32_t *k2d_static_ptr[64];     // device address of the array on each device, filled on first use

int k2d_step_discrete(k2d_state *s, const int32_t *dev_actions, int32_t n_steps, float *dev_reward, uint8_t *dev_done) {
    if (!s || !dev_actions || !dev_reward || !dev_done) return K2D_ERR_NULL;
    if (n_steps < 1 || n_steps > s->cfg.max_fused_steps) return K2D_ERR_STEPS;
    if (((uintptr_t)dev_actions & 3) || ((uintptr_t)dev_reward & 3)) return K2D_ERR_ALIGN;
    CUDA_OK(cudaSetDevice(s->cfg.device));
    StepParams prm = step_params(s, reinterpret_cast<const float *>(dev_actions), n_steps, dev_reward, dev_done, s->dev_scratch, 1);
    CUDA_OK(order_envs(s, prm));
    CUDA_OK(K2D_DISPATCH(launch_step, s, s, prm));
    return K2D_OK;
}

int k2d_step_static_scratch(k2d_state *s, const float *dev_actions, int32_t n_steps, float *dev_reward, uint8_t *dev_done) {
    if (!s || !dev_actions || !dev_reward || !dev_done) return K2D_ERR_NULL;
    if (n_steps < 1 || n_steps > s->cfg.max_fused_steps) return K2D_ERR_STEPS;
    if (((uintptr_t)dev_actions & 3) || ((uintptr_t)dev_reward & 3)) return K2D_ERR_ALIGN;
    const k2d_config &c = s->cfg;
    if (c.n_envs > K2D_STATIC_SCRATCH_MAX_ENVS || s->groups > K2D_STATIC_SCRATCH_MAX_ENVS || c.device >= 64) {
        std::fprintf(stderr, "k2d_step_static_scratch: n_envs = %d is beyond the built-in scratch (at most %d envs); use k2d_step\n",
                     c.n_envs, K2D_STATIC_SCRATCH_MAX_ENVS);
        return K2D_ERR_LIMIT;
    }
    CUDA_OK(cudaSetDevice(c.device));
    uint32_t *scratch = nullptr;
    {
        // In host code the array's name is only a handle; the kernel needs its address on this device.
        std::lock_guard<std::mutex> lock(k2d_static_mutex);
        if (!k2d_static_ptr[c.device]) {
            void *p = nullptr;
            CUDA_OK(cudaGetSymbolAddress(&p, k2d_static_scratch));
            k2d_static_ptr[c.device] = (uint32_t *)p;
        }
        scratch = k2d_static_ptr[c.device];
    }
    const StepParams prm = step_params(s, dev_actions, n_steps, dev_reward, dev_done, scratch);
    // a launch never has more scene groups than envs rounded up to a whole block, so the limit on n_envs bounds the scratch slots
    CUDA_OK(K2D_DISPATCH(launch_step, s, s, prm));
    return K2D_OK;
}

int k2d_measure_fp32_peak(int32_t device, float *dev_scratch, size_t scratch_floats, float *host_tflops) {
    if (!dev_scratch || !host_tflops) return K2D_ERR_NULL;
    CUDA_OK(cudaSetDevice(device));
    int num_sms = 0;
    CUDA_OK(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, device));
    const int threads = 256, blocks = num_sms * 8;        // 2048 threads per SM: every scheduler has chains to pick from
    if (scratch_floats < (size_t)threads * blocks) return K2D_ERR_ARG;
    cudaEvent_t e0, e1;
    CUDA_OK(cudaEventCreate(&e0));
    CUDA_OK(cudaEventCreate(&e1));
    float best_ms = 0.0f;
    for (int rep = 0; rep < 5; ++rep) {       // the first launches warm up; the best of the rest counts
        CUDA_OK(cudaEventRecord(e0, 0));
        k2d_fma_chain_kernel<<<blocks, threads>>>(dev_scratch, 0.999f, 1e-3f);
        CUDA_OK(cudaEventRecord(e1, 0));
        CUDA_OK(cudaEventSynchronize(e1));
        float ms = 0.0f;
        CUDA_OK(cudaEventElapsedTime(&ms, e0, e1));
        if (rep >= 2 && (best_ms == 0.0f || ms < best_ms)) best_ms = ms;
    }
    CUDA_OK(cudaEventDestroy(e0));
    CUDA_OK(cudaEventDestroy(e1));
    const double flops = 2.0 * kFmaChainSteps * kFmaChains * (double)threads * blocks;
    *host_tflops = (float)(flops / (best_ms * 1e-3) / 1e12);
    return K2D_OK;
}

const char *k2d_error_string(int code) {
    switch (code) {
        case K2D_OK: return "ok";
        case K2D_ERR_NULL: return "null pointer";
        case K2D_ERR_CONFIG: return "invalid config";
        case K2D_ERR_ALIGN: return "misaligned device pointer";
        case K2D_ERR_LEVEL: return "invalid level data";
        case K2D_ERR_STEPS: return "n_steps out of range";
        case K2D_ERR_CUDA: return "CUDA runtime error";
        case K2D_ERR_ARG: return "invalid argument";
        case K2D_ERR_LIMIT: return "size beyond a built-in limit";
        case K2D_ERR_CHECK: return "an index check of the checked build failed";
        case K2D_ERR_BUILD: return "this build of the library does not have that feature compiled in";
        case K2D_ERR_WAIT: return "a scene group gave up waiting for another; the last step is incomplete";
        default: return "unknown error";
    }
}

void k2d_destroy(k2d_state *s) { delete s; }

}  // extern "C"
