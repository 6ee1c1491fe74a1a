/*
 * k2d.h -- C ABI of the batched 2D rigid-body environment step (sm_100a CUDA library).
 *
 * The library advances thousands of independent fixed-size scenes of the Kinetix / Jax2D
 * kind (arxiv 2410.23208): circles, convex polygons of 3 or 4 vertices, revolute joints with
 * motors, thrusters.  One call of k2d_step runs, for every scene and for n_steps steps, the
 * paper's Algorithm 1 (gravity, collision manifolds, motors, thrusters, warm start, a fixed
 * number of sequential-impulse solver iterations over joints (revolute, fixed, with rotation
 * limits) then contacts, Euler step),
 * followed by Kinetix's touch reward / termination ("Reward" paragraph: green touches blue
 * = +1 and done, green touches red = -1 and done) and the auto-reset.
 *
 * Conventions
 *  - C99 types only; every function returns int: 0 = K2D_OK, negative = error, and on error
 *    no device work has been enqueued.
 *  - The CALLER owns every device buffer and the CUDA stream.  The library owns only the host
 *    handle; it never allocates or frees device memory.  k2d_step and k2d_obs are asynchronous
 *    on the stream given in the config; k2d_create, k2d_reset, k2d_get_state, k2d_set_state
 *    and k2d_status synchronise that stream.
 *  - "dev_" pointers are device memory on the config's device; the state buffer and the level pool
 *    must be 16-byte aligned, every other device pointer 4-byte aligned.  "host_" pointers are host
 *    memory.  Every call that touches the device makes the config's device current (cudaSetDevice)
 *    and leaves it current, so handles on several devices can be used from one thread.
 *  - Shape index inside a scene: polygons 0 .. n_polygons-1, then circles.  Pair order (used by
 *    the solver and by the accumulated-impulse slots): polygon-polygon pairs (i<j,
 *    lexicographic), polygon-circle pairs (polygon major), circle-circle pairs (i<j);
 *    polygon-polygon pairs own two manifold slots, the others one.
 *  - All floating point is IEEE binary32.  Results are bit-reproducible from run to run and
 *    do not depend on n_envs, on lanes_per_scene or on how many steps are fused per call.
 */
#ifndef K2D_H_
#define K2D_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define K2D_OK 0
#define K2D_ERR_NULL (-1)          /* a required pointer is null                         */
#define K2D_ERR_CONFIG (-2)        /* a config field is out of range                     */
#define K2D_ERR_ALIGN (-3)         /* a device pointer is not aligned as required        */
#define K2D_ERR_LEVEL (-4)         /* level data invalid (non-finite, bad index, ...)    */
#define K2D_ERR_STEPS (-5)         /* n_steps < 1 or > max_fused_steps                   */
#define K2D_ERR_CUDA (-6)          /* a CUDA runtime call failed                         */
#define K2D_ERR_ARG (-7)           /* another argument is invalid                        */
#define K2D_ERR_LIMIT (-8)         /* a size is beyond a limit built into the library    */
#define K2D_ERR_WAIT (-9)          /* k2d_status: a wait inside k2d_step ran out (see there) */
#define K2D_ERR_CHECK (-10)        /* k2d_status of a checked build: an index was out of range    */
#define K2D_ERR_BUILD (-11)        /* the call needs a build of the library with another compile flag */

#define K2D_MAX_POLYGONS 12
#define K2D_MAX_CIRCLES 4
#define K2D_MAX_SHAPES 16
#define K2D_MAX_JOINTS 6
#define K2D_MAX_THRUSTERS 2

#define K2D_RESET_NONE 0           /* keep stepping; flags are reported every step they hold */
#define K2D_RESET_SAME_LEVEL 1     /* on done, the env restarts on its own level              */
#define K2D_RESET_POOL 2           /* on done, level = hash(seed, env, episode) mod n_levels  */

#define K2D_ROLE_NONE 0
#define K2D_ROLE_GREEN 1
#define K2D_ROLE_BLUE 2
#define K2D_ROLE_RED 3

#define K2D_STATUS_NONFINITE 1     /* per-env status bit: the state became non-finite         */

/* Engine and environment parameters.  The paper leaves dt, the iteration count and the
 * correction coefficients open; the defaults written by k2d_default_config are dt = 1/60,
 * gravity_y = -9.81, 8 solver iterations, contact_alpha = joint_alpha = 6 /s,
 * contact_beta = joint_beta = 0.1, joint_gamma = 6 /s, slop = 0.005 m,
 * restitution_threshold = 1 m/s, face_tol = 1e-3 m, motor_rho = 1, aabb_margin = 0.01 m, warm starting on. */
/* solver_batch (paper, "Parallelised Computation and Batched Impulse Resolution"): the scene's manifold slots (two per
 * polygon pair, one per other pair) are cut into ceil(n_slots / B) batches.  In every solver iteration, after the joints,
 * the batches are solved one after the other; the rows of one batch are all solved against the velocities the batch
 * starts with and applied together afterwards (in canonical order).  The active manifolds are spread over as many batches
 * as possible: the i-th active manifold in canonical order goes to batch i mod n_batches.  While a scene has no more
 * active manifolds than batches this is the sequential solve, bit for bit; the paper's default is B = 16.  The library
 * runs this mode on its general, untuned path (constraint rows in the scratch tail); it is there for fidelity. */
typedef struct k2d_config {
    int32_t n_envs;                /* >= 1                                                      */
    int32_t n_polygons;            /* 1 .. K2D_MAX_POLYGONS                                     */
    int32_t n_circles;             /* 0 .. K2D_MAX_CIRCLES                                      */
    int32_t n_joints;              /* 0 .. K2D_MAX_JOINTS                                       */
    int32_t n_thrusters;           /* 0 .. K2D_MAX_THRUSTERS                                    */
    int32_t n_actions;             /* >= 1; bindings index into the action row                  */
    int32_t n_levels;              /* >= 1, size of the level pool                              */
    int32_t solver_iters;          /* >= 0                                                      */
    int32_t warm_start;            /* 0 / 1 (paper: "Impulse Accumulation and Warm Starting")   */
    int32_t auto_reset;            /* K2D_RESET_*                                               */
    int32_t max_episode_steps;     /* 0 = no horizon; else done when step_count reaches it      */
    int32_t max_fused_steps;       /* largest n_steps k2d_step accepts                          */
    int32_t frame_skip;            /* >= 1: engine steps each action row is held for (paper: 2)  */
    float dt, gravity_y;
    float contact_alpha;           /* velocity correction: bias = alpha * max(pen - slop, 0)    */
    float contact_beta;            /* positional correction: beta * max(pen - slop, 0)          */
    float slop;
    float restitution_threshold;   /* approach speed below which a contact does not bounce      */
    float face_tol;                /* polygon-polygon reference face hysteresis                 */
    float joint_alpha, joint_beta; /* the same two corrections for the joint's point constraint */
    float motor_rho;               /* rho of the motor law j = p tanh((wa - wb - s A) rho)      */
    float aabb_margin;             /* bounding boxes further apart than this skip narrowphase   */
    float joint_gamma;             /* angular correction of fixed joints and joint limits: gamma * angle error */
    float dense_kappa;             /* dense reward kappa * (d_t - d_t+1), d = green-blue distance; 0 = off */
    uint64_t seed;                 /* seed of the K2D_RESET_POOL hash                           */
    int64_t env_offset;            /* global index of env 0 (sharding over several GPUs)        */
    int32_t device;                /* CUDA device ordinal                                       */
    int32_t lanes_per_scene;       /* 0 = library default (32 for few envs, else 16); or 8, 16, 32 */
    int32_t solver_batch;          /* 0 = contacts solved one after the other (default); B > 0 = the paper's batched solve, see below */
    int32_t reserved;              /* 0 */
    void *cuda_stream;             /* cudaStream_t of the caller (NULL = default stream)        */
} k2d_config;

/* One scene as the caller describes it.  Entities beyond the config's counts are ignored.
 * Polygon vertices are in the body frame, counter-clockwise, with the centroid at the origin
 * (|centroid| <= 1e-3 x extent is enforced).  Mass and inertia follow from density (uniform
 * lamina); is_static shapes have infinite mass (paper: fixated shapes). */
typedef struct k2d_level {
    float poly_verts[K2D_MAX_POLYGONS][4][2];
    int32_t poly_nverts[K2D_MAX_POLYGONS];           /* 3 or 4                                  */
    float circle_radius[K2D_MAX_CIRCLES];
    float pos[K2D_MAX_SHAPES][2], angle[K2D_MAX_SHAPES];      /* initial pose                   */
    float vel[K2D_MAX_SHAPES][2], angvel[K2D_MAX_SHAPES];     /* initial velocity               */
    float density[K2D_MAX_SHAPES], friction[K2D_MAX_SHAPES], restitution[K2D_MAX_SHAPES];
    int32_t is_static[K2D_MAX_SHAPES], role[K2D_MAX_SHAPES], active[K2D_MAX_SHAPES];
    int32_t joint_a[K2D_MAX_JOINTS], joint_b[K2D_MAX_JOINTS]; /* shape indices                  */
    float joint_anchor_a[K2D_MAX_JOINTS][2], joint_anchor_b[K2D_MAX_JOINTS][2]; /* body frame   */
    float motor_speed[K2D_MAX_JOINTS], motor_power[K2D_MAX_JOINTS];
    int32_t motor_binding[K2D_MAX_JOINTS], joint_active[K2D_MAX_JOINTS];
    /* paper, "Fixed Joints" / "Joint Limits"; the relative rotation of a joint is angle[a] - angle[b] */
    int32_t joint_fixed[K2D_MAX_JOINTS];             /* 1: also holds the relative rotation at joint_fixed_angle */
    int32_t joint_limited[K2D_MAX_JOINTS];           /* 1: revolute, relative rotation kept in [min, max]       */
    float joint_fixed_angle[K2D_MAX_JOINTS], joint_min[K2D_MAX_JOINTS], joint_max[K2D_MAX_JOINTS];
    int32_t thr_shape[K2D_MAX_THRUSTERS];
    float thr_pos[K2D_MAX_THRUSTERS][2], thr_rot[K2D_MAX_THRUSTERS], thr_power[K2D_MAX_THRUSTERS];
    int32_t thr_binding[K2D_MAX_THRUSTERS], thr_active[K2D_MAX_THRUSTERS];
} k2d_level;

typedef struct k2d_state k2d_state;   /* opaque host handle */

/* Fills *cfg with the defaults listed above for the given scene dimensions (n_actions =
 * n_joints + n_thrusters, n_levels = n_envs, auto_reset = NONE, max_fused_steps = 64,
 * frame_skip = 1). */
int k2d_default_config(k2d_config *cfg, int32_t n_envs, int32_t n_polygons, int32_t n_circles,
                       int32_t n_joints, int32_t n_thrusters);

/* Bytes of device memory the caller must provide for the state buffer (scene state of all
 * envs, a small control block, and the solver's overflow scratch) and for the level pool.
 * Host-only; 0 on an invalid config. */
size_t k2d_state_bytes(const k2d_config *cfg);
size_t k2d_level_pool_bytes(const k2d_config *cfg);
/* The state buffer without its overflow-scratch tail, which is its last part: what a caller who steps only
 * through k2d_step_static_scratch (below) has to provide.  A handle created over a buffer of this size must
 * never be given to k2d_step or k2d_step_discrete, which write the tail.  Host-only; 0 on an invalid config. */
size_t k2d_state_bytes_no_scratch(const k2d_config *cfg);

/* Validates the config and the n_levels host levels, derives mass properties and the pair
 * collision mask (joined shapes do not collide: paper, "Joints"), uploads the level pool to
 * dev_level_pool_buf, resets every env (env i on level i mod n_levels) and returns a handle.
 * Both buffers stay owned by the caller and must outlive the handle. */
int k2d_create(const k2d_config *cfg, void *dev_state_buf, void *dev_level_pool_buf,
               const k2d_level *host_levels, k2d_state **out);

/* Restarts every env: env i on level host_level_ids[i] (NULL: i mod n_levels), episode 0,
 * zero accumulated impulses, zero counters. */
int k2d_reset(k2d_state *s, const int32_t *host_level_ids);

/* Advances every env by n_steps steps (paper, Algorithm 1 + "Reward").  dev_actions is
 * [ceil(n_steps / frame_skip)][n_envs][n_actions] floats, one row per frame_skip steps of this
 * call (frame_skip = 1: one row consumed per step; the paper trains with a frame skip of 2;
 * reward and done are still written for every engine step) (motor actions are clipped
 * to [-1, 1], thruster actions to [0, 1]: paper, "Action Space"); dev_reward [n_steps][n_envs]
 * floats in {-1, 0, +1}, plus, if dense_kappa is not 0, the paper's auxiliary dense reward
 * kappa * (d_t - d_t+1) with d the distance between the positions of the first green and the
 * first blue shape before and after the step; dev_done [n_steps][n_envs] bytes.  1 <= n_steps <= max_fused_steps.
 * The whole call is one kernel launch; scene state stays on chip between the fused steps. */
int k2d_step(k2d_state *s, const float *dev_actions, int32_t n_steps, float *dev_reward, uint8_t *dev_done);

/* The same step with the paper's multi-discrete action space ("Action Space": every motor and
 * thruster is inactive or at maximum power, motors forwards or backwards): dev_actions is
 * [ceil(n_steps / frame_skip)][n_envs][n_actions] int32 codes (one row per frame_skip steps, as for k2d_step); a motor reads 0 = off, 1 = forwards (+1), 2 = backwards
 * (-1), anything else off; a thruster reads 0 = off, anything else on. */
int k2d_step_discrete(k2d_state *s, const int32_t *dev_actions, int32_t n_steps, float *dev_reward, uint8_t *dev_done);

/* The paper has no counterpart of this call; it exists for one kind of user of this library.
 * k2d_step keeps the contact records of a very crowded scene (far more touching pairs than
 * lanes working on the scene) in the scratch tail of the state buffer, which the caller has to
 * allocate.  Some callers cannot: a process whose device memory is one arena fixed at start-up,
 * a plug-in handed a pre-sized buffer by its host, code running where cudaMalloc is forbidden
 * (a real-time loop).  For them this variant does exactly what k2d_step does, with the same
 * arguments and bit-identical results, but keeps those records in an array compiled into the
 * library (K2D_STATIC_SCRATCH_MAX_ENVS x 13920 bytes, about 14 MB, resident on every GPU that
 * loads the library until the process exits) and never touches the scratch tail.  It allocates
 * and frees nothing, on the host side of CUDA or on the device.
 *  - n_envs above K2D_STATIC_SCRATCH_MAX_ENVS is refused with K2D_ERR_LIMIT (and a line on
 *    stderr); nothing is enqueued.
 *  - The first call on each device looks up the array's device address (with that device made
 *    current); make that first call before any stream capture begins.
 *  - All handles and streams of a process share the one array per device.  Nothing in it has
 *    to start at zero (every record is written before it is read), so calls one after another
 *    need no clearing; calls that overlap on the GPU (two streams, two handles) race on it
 *    and must be serialised by the caller. */
#define K2D_STATIC_SCRATCH_MAX_ENVS 1024
int k2d_step_static_scratch(k2d_state *s, const float *dev_actions, int32_t n_steps, float *dev_reward, uint8_t *dev_done);

/* Symbolic per-entity observation (paper, tables "Information provided for shapes / joints /
 * thrusters"): dev_obs is [n_envs][k2d_obs_floats] floats; per env the shape rows (29 floats
 * each), two rows per joint (11 + n_actions floats each), one row per thruster (6 floats).
 * The buffer is plain row-major, so the same memory read as [n_envs][k2d_obs_floats] is the
 * paper's Symbolic-Flat observation (the rows concatenated). */
int k2d_obs(k2d_state *s, float *dev_obs);
int k2d_obs_floats(const k2d_config *cfg);

/* k2d_step followed by k2d_obs of the state it leaves, as one kernel launch: the group of lanes that has stepped an env
 * writes the env's observation rows from shared memory before it moves on, so the state is not read back from memory
 * by a second kernel.  This is the call for a training loop that takes one engine step (or one frame-skip window) and
 * one observation at a time (paper, "Kinetix": step, then the Symbolic-Entity observation).  Same arguments as k2d_step
 * plus dev_obs as for k2d_obs; results identical to the two separate calls. */
int k2d_step_obs(k2d_state *s, const float *dev_actions, int32_t n_steps, float *dev_reward, uint8_t *dev_done, float *dev_obs);

/* Pixel observation (paper: the "Pixels" observation space, a 125 x 125 image; the paper gives
 * no more than the size).  dev_pixels is [n_envs][K2D_PIXELS][K2D_PIXELS][4] bytes, RGBA, row 0
 * at the top, 4-byte aligned.  The centre of pixel (row r, column c) is the world point
 * x = -3.125 + (c + 0.5) * 0.05, y = 5.75 - (r + 0.5) * 0.05.  A pixel has the colour of the
 * highest-index active shape whose interior or boundary contains its centre, white otherwise:
 * green (0, 200, 0), blue (0, 0, 220), red (220, 0, 0), no role (128, 128, 128) or, if fixated,
 * (64, 64, 64); alpha is 255.  Joints and thrusters are not drawn.  Asynchronous on the stream. */
#define K2D_PIXELS 125
int k2d_render(k2d_state *s, uint8_t *dev_pixels);

/* Canonical host copy of the dynamic state, for checkpoints and comparisons: per env
 * k2d_canonical_words 4-byte words: pos[N][2], angle[N], vel[N][2], angvel[N] (floats),
 * acc[n_slots][2] (accumulated normal, tangent impulse per manifold slot), jacc[n_joints][3]
 * (accumulated impulse of the joint's point constraint x, y and of a fixed joint's angular row),
 * then int32 step_count, episode_count, level_id, status.  set_state followed by k2d_step
 * continues bit-identically. */
int k2d_canonical_words(const k2d_config *cfg);
int k2d_get_state(k2d_state *s, void *host_canonical);
int k2d_set_state(k2d_state *s, const void *host_canonical);

/* host_counts[8] (int64), all since the last k2d_reset: non-finite events, auto-resets, active
 * manifolds summed over env-steps, env-steps, pairs that passed the bounding-box test (polygon-
 * polygon, polygon-circle, circle-circle), pairs with at least one active manifold.
 * Returns K2D_ERR_WAIT (with the counts filled in) if, in some k2d_step since the last k2d_reset,
 * a group of lanes waited longer than its limit (seconds) for another group to finish an earlier
 * part of the same env's steps: the kernel then gave up on that env instead of hanging, and the
 * states are not valid any more; k2d_reset clears the condition. */
int k2d_status(k2d_state *s, int64_t *host_counts);

/* Host only, no device needed: validates one level against the config and returns the constants
 * the library derives from it: inv_mass[N], inv_inertia[N] (floats; 0 for fixated or absent shapes)
 * and collide[n_pairs] (bytes; pair order as above).  Any output pointer may be NULL. */
int k2d_level_info(const k2d_config *cfg, const k2d_level *host_level, float *host_inv_mass, float *host_inv_inertia,
                   uint8_t *host_collide);

/* Debug aid: when dev_trace is non-null every later step also writes the manifolds of each
 * env's latest step to dev_trace[n_envs][n_slots][6] = px, py, nx, ny, penetration, active
 * (slots indexed in the library's internal size class, see k2d_trace_slots). */
int k2d_set_trace(k2d_state *s, float *dev_trace);
int k2d_trace_slots(const k2d_state *s);

/* 1 if the library was compiled with -DK2D_CHECKED, else 0.  The checked build compares every index its kernels unpack
 * from packed words or read from tables (bodies, pairs, memory records, level ids, warm entries, solver levels, scratch
 * slots, counts) with its limit; a violation is recorded (k2d_status then returns K2D_ERR_CHECK until the next
 * k2d_reset) and the access is redirected to index 0; nothing traps.  It stands in for a memory checker. */
int k2d_is_checked_build(void);

/* Host-side facts about a handle's launches.  k2d_resident_groups: scenes the device steps at once for this handle (with
 * more envs than that a launch goes through a work queue, and from one and a half times as many on it first sorts the envs
 * by what their steps cost, in two small launches of its own; launches of fewer than 8 steps reuse that order 16 times).  k2d_lanes_per_scene: 8, 16 or 32.
 * k2d_step_launches: kernel launches that the next k2d_step, k2d_step_discrete or k2d_step_obs call with n_steps steps
 * makes (1 or 3; k2d_step_obs one more for scenes whose observation does not fit beside the scene in shared memory). */
int k2d_resident_groups(const k2d_state *s);
int k2d_lanes_per_scene(const k2d_state *s);
int k2d_step_launches(const k2d_state *s, int32_t n_steps);
/* Test aid: the work items ((run of 8 steps, env) pairs) that one ticket of a launch's work queue stands for: the scene
 * groups of the warps that step in lockstep (10 for L scenes on a full device). */
int k2d_items_per_ticket(const k2d_state *s);

/* Measurement aid.  In a library compiled with -DK2D_PHASE_CLOCKS the step kernel adds up, per phase of an environment
 * step (Algorithm 1's stages as this library cuts them), the SM cycles that every scene group spends in it.  The call waits
 * for the handle's stream, copies the first n (<= K2D_PHASES) sums to host_cycles and clears them.  Order of the phases:
 * world geometry and boxes; motors and thrusters; joint pre-step; box test; narrowphase; contact pre-step (records);
 * solver levels; warm start; solver iterations; Euler step and positional corrections; reward / done / reset; the whole
 * contact solve of scenes on the memory-record path; state load; state store.  In any other build: zeros and K2D_ERR_BUILD. */
#define K2D_PHASES 14
int k2d_phase_cycles(k2d_state *s, uint64_t *host_cycles, int32_t n);

/* Test aid.  With more envs than the device holds scene groups, k2d_step hands out runs of 8 steps of an env to whichever
 * group is free; a group that gets a later run of an env before the earlier one is back in memory polls for it, about
 * every 100 ns, at most `polls` times (default 2^24, a few seconds; values below 64 are raised to 64), then records
 * K2D_ERR_WAIT for k2d_status and gives up.  A small limit lets a test make that wait run out. */
int k2d_set_wait_limit(k2d_state *s, uint32_t polls);

/* Evaluates the library's own sine/cosine and tanh routines on n device floats (the step
 * uses these instead of libm so that results are reproducible bit for bit). */
int k2d_eval_sincos_tanh(const float *dev_x, int32_t n, float *dev_cos, float *dev_sin, float *dev_tanh, void *cuda_stream);

/* Measurement aid, not part of the step: runs chains of dependent fused multiply-adds on every SM of the device (eight
 * independent chains per thread, 2048 threads per SM) on the default stream and returns the FP32 rate they reach, in
 * TFLOP/s (a multiply-add counts 2), in *host_tflops: the measured counterpart of SMs x 128 lanes x 2 x clock.
 * dev_scratch: at least 2048 x the device's SM count floats of device memory (overwritten).  Synchronous. */
int k2d_measure_fp32_peak(int32_t device, float *dev_scratch, size_t scratch_floats, float *host_tflops);

const char *k2d_error_string(int code);
void k2d_destroy(k2d_state *s);

#ifdef __cplusplus
}
#endif
#endif /* K2D_H_ */
