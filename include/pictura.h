/*
 * pictura.h -- C ABI of the batched egocentric rasterizer (CUDA, sm_100a).
 *
 * The library renders, for every agent of every environment and every camera of an ego-mounted
 * rig, a semantic-class image (u8) and a depth image (IEEE binary16) of the agent's surroundings:
 * the triangles of the environment's map and the other agents as oriented 3-D boxes, under a
 * pinhole projection with a z-buffer.  This is the rasterizer Phi of the paper (Sec. 3.2, Eq. 2:
 * I_{i,k} = Phi(A_i, W_i, K_{i,k}); "only the surroundings are rendered"), with a class/depth
 * output in place of the paper's shaded colour.
 *
 * Conventions (paper, table "Camera rig"): world z up; agent frame x forward, y left, z up; yaw
 * counter-clockwise about z; a camera is mounted at `mount` in the agent frame, turned by `yaw`
 * about z and pitched up by `pitch`; intrinsics are focal lengths in pixels with the principal
 * point at the image centre.  Pixel (u, v) -- column u left to right, row v top to bottom,
 * row-major storage -- samples the ray through (u + 0.5, v + 0.5).
 *
 * Per pixel: a primitive covers the pixel when the ray hits it (edge functions with a top-left
 * fill rule on exact zeros, no geometric clipping); its depth z is the distance along the optical
 * axis; fragments with near <= z <= far are kept; the smallest z wins, exact ties go to the lower
 * primitive index (map triangles in the order given, then 12 triangles per agent box).  Pixels
 * without a fragment show the analytic ground plane z = 0 (ground class, depth min(far, hit
 * depth)) below the horizon and sky (sky class, depth far) above it.  An agent never sees its own
 * box; agents of other environments are never visible; an inactive agent is not drawn and its
 * own images are sky/far.  Arithmetic is float32; results agree with a double-precision
 * evaluation except at pixels whose edge function, depth gap or clip plane is within 1e-5
 * relative of a decision boundary.
 *
 * Memory: every pointer marked "dev" is device memory of the scene's CUDA device, owned by the
 * caller; "host" pointers are ordinary host memory.  The library never takes ownership of a
 * caller's buffer.  Unless stated otherwise calls are asynchronous on the given CUDA stream
 * (a cudaStream_t passed as void*; NULL is the default stream) and allocate nothing.
 *
 * One stream at a time per scene: every pic_render / pic_step / pic_set_state of a scene writes
 * the scene's own per-call buffers (agent geometry, per-view cameras, per-camera tables, the
 * survivor lists handed from the cull kernel to the render kernel, the list of left-out tiles,
 * timing events), and options are plain fields read when a call is issued.  Calls on one scene
 * must therefore be issued from one host thread at a time and be ordered on the device -- the
 * same stream, or streams ordered with events; two calls of one scene that overlap on the GPU
 * race silently.  Different scenes are independent.
 *
 * Errors: every call returns a pic_status; nothing throws, aborts or traps.  pic_last_error()
 * returns a thread-local description of the last failure.  Device-detected conditions are
 * accumulated in sticky flags read by pic_get_status().
 */
#ifndef PICTURA_H
#define PICTURA_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pic_scene pic_scene; /* opaque; created and destroyed by the library */

typedef enum {
    PIC_OK = 0,
    PIC_ERR_INVALID_ARG = 1, /* NULL where a pointer is required, bad struct size, bad device  */
    PIC_ERR_SHAPE = 2,       /* non-positive or unsupported sizes, inconsistent offsets        */
    PIC_ERR_OOM = 3,         /* host or device allocation failed                                */
    PIC_ERR_CUDA = 4,        /* a CUDA runtime call failed (see pic_last_error)                 */
    PIC_ERR_CAPACITY = 5,    /* a fixed-size entry point was given more than it can hold        */
    PIC_ERR_NONFINITE = 6    /* reserved for status flags                                       */
} pic_status;

/* Sticky device flags returned by pic_get_status. */
#define PIC_FLAG_NONFINITE_POSE 0x1u /* a pose, size or action was NaN/Inf (or a step overflowed): that agent is treated as
                                        inactive for the call -- its images are sky, nobody sees it -- and pic_step leaves
                                        its state as it was */
#define PIC_FLAG_COLOUR_INCOMPLETE 0x2u /* pic_render_rgb: a 64 x 64 tile saw more primitives than its list holds (254) and shows
                                           only the background */
#define PIC_FLAG_COLOUR_FRAGMENTS 0x4u  /* pic_render_rgb, antialiased: one pixel held more than 1023 partially covering
                                           fragments in front of its opaque surface; the surplus was dropped */

/* One pinhole camera of the rig, in the agent frame (x forward, y left, z up). */
typedef struct {
    float mount_x, mount_y, mount_z; /* metres                                                   */
    float yaw;                       /* rad, counter-clockwise about z (left positive)           */
    float pitch;                     /* rad, up positive; no roll                                */
    float fx, fy;                    /* focal lengths in pixels: fx = (W/2)/tan(hfov/2), same for fy */
} pic_camera;

typedef struct {
    uint32_t size;                 /* = sizeof(pic_scene_desc); rejects mismatched headers       */
    int32_t E, A, K, H, W;         /* environments, agents/env, cameras/agent, image rows, cols  */
    float near_z, far_z;           /* kept depth range, metres, 0 < near_z < far_z              */
    int32_t num_maps;              /* M >= 1 maps                                                */
    const int32_t* env_map_id;     /* host [E], values in [0,M); NULL: identity if M == E, else all 0 */
    const int64_t* map_tri_offset; /* host [M+1], non-decreasing, [0] == 0                       */
    const float* tri_xyz;          /* host [N,3,3] f32 world coordinates, N = map_tri_offset[M] */
    const uint8_t* tri_class;      /* host [N] class id of each triangle                         */
                                   /* (both arrays must be HOST memory in this build: the hierarchy is built on
                                      the host; device pointers are not accepted)                              */
    uint8_t agent_class;           /* class written for agent boxes                              */
    uint8_t sky_class;             /* background above the horizon                               */
    uint8_t ground_class;          /* background below the horizon                               */
    uint8_t reserved;
    int32_t device;                /* CUDA device ordinal                                        */
    const float* tri_vis_cos;      /* host [N] or NULL: 0 = ordinary two-sided triangle; c in (0, 1] = the triangle
                                      is drawn in a view only from its front side (normal (V1-V0)x(V2-V0)) and only if
                                      the direction from its centroid to the camera is within acos(c) of that normal --
                                      the paper's traffic-light disks "visible only within a limited angular range"
                                      (Sec. 3.2), given as triangle fans.  Such triangles are never paired into quads. */
} pic_scene_desc;

/*
 * Build a scene: copies the map (the caller may free its arrays on return), builds the per-map
 * culling hierarchy and allocates all device memory the scene will ever need, including the
 * kinematic state [E,A,4] used by pic_step.  Synchronous.  At most 2^24 - 12*A triangles per map.
 */
pic_status pic_scene_create(const pic_scene_desc* desc, pic_scene** out);

/* Free a scene and everything it owns.  Synchronises the device.  NULL is accepted. */
pic_status pic_scene_destroy(pic_scene* scene);

/*
 * Render all E*A*K views (the rasterizer Phi, Eq. 2).
 *   poses      dev f32 [E,A,3]   x, y, yaw of each agent (box centre on the ground plane)
 *   dims       dev f32 [E,A,3]   box length (along heading), width, height
 *   active     dev u8  [E,A] or NULL (all active)
 *   rig        host    [K]       copied during the call
 *   out_class  dev u8  [E,A,K,H,W]
 *   out_depth  dev u16 [E,A,K,H,W] binary16 bit patterns
 * out_class must be 16-byte aligned and out_depth 16-byte aligned.
 */
pic_status pic_render(pic_scene* scene, const float* poses, const float* dims, const uint8_t* active,
                      const pic_camera* rig, uint8_t* out_class, uint16_t* out_depth, void* cuda_stream);

/*
 * Same as pic_render with HOST inputs and outputs: copies poses/dims/active to the device, renders
 * into staging buffers owned by the scene (allocated on first use: 3*E*A*K*H*W bytes) and copies
 * both images back.  Returns after the copies completed (the stream is synchronised).  Host
 * buffers may be pageable or pinned; pinned is faster.
 */
pic_status pic_render_host(pic_scene* scene, const float* poses, const float* dims, const uint8_t* active,
                           const pic_camera* rig, uint8_t* out_class, uint16_t* out_depth, void* cuda_stream);

/*
 * Kinematic state for pic_step: state dev f32 [E,A,4] = x, y, yaw, v; dims and active as in
 * pic_render (copied into the scene).  pic_get_state copies the state out to dev memory.
 */
pic_status pic_set_state(pic_scene* scene, const float* state, const float* dims, const uint8_t* active,
                         void* cuda_stream);
pic_status pic_get_state(pic_scene* scene, float* state_out, void* cuda_stream);

/*
 * Class of each agent's box (Sec. 3.2: pedestrians, cyclists and vehicles each in its own hue): classes dev u8
 * [E,A], copied into the scene on `cuda_stream`; NULL returns to desc.agent_class for every agent.  Used by all
 * later pic_render / pic_step calls.
 */
pic_status pic_set_agent_classes(pic_scene* scene, const uint8_t* classes, void* cuda_stream);

/*
 * One simulator step: explicit-Euler kinematic bicycle update of every active agent, everything
 * computed from the old state,
 *     x += v cos(yaw) dt,  y += v sin(yaw) dt,  yaw += (v / wheelbase) tan(steer) dt,
 *     v = clamp(v + accel dt, 0, v_max)            (dt 0.1 s, wheelbase 2.8 m, v_max 30 m/s),
 * then a render of all views from the NEW state (the paper's loop: each agent acts, then is
 * rendered for its neighbours, Sec. 1; its own dynamics use jerk actions and are not reproduced).
 *   actions    dev f32 [E,A,2]   accel (m/s^2), steer (rad)
 */
pic_status pic_step(pic_scene* scene, const float* actions, const pic_camera* rig, uint8_t* out_class,
                    uint16_t* out_depth, void* cuda_stream);

/* Synchronise `cuda_stream`, then read and clear the sticky device flags (PIC_FLAG_*) into *flags (host). */
pic_status pic_get_status(pic_scene* scene, uint32_t* flags, void* cuda_stream);

/*
 * Options (all default 0):
 *   PIC_OPT_BRUTE_FORCE   1: render with the exhaustive kernel (every primitive against every
 *                         pixel tile, no culling hierarchy) -- a slow cross-check that shares the
 *                         per-primitive arithmetic with the production kernel.
 *   PIC_OPT_DEPTH32       value = dev f32* [E,A,K,H,W] (as uintptr) or 0: also write the float32
 *                         depth the binary16 image was rounded from.
 *   PIC_OPT_COUNTERS      value = dev u64* [16] (as uintptr) or 0: accumulate work counters (tiles,
 *                         group tests, leaf tests, primitives tested, set up, rasterized by their
 *                         thread, records, record-list overflows, records classified per cell (once
 *                         per 16-row strip they reach), cells visited, tiles rendered by the
 *                         cooperative kernel).
 *   PIC_OPT_VIEW_FIRST,   render only views [first, first + count) (flat index (e*A + a)*K + k);
 *   PIC_OPT_VIEW_COUNT    count 0 = through the last view.  Other views' pixels are left untouched.
 *   PIC_OPT_OCCLUSION     value = dev u32* [E,A,K,A,2] (as uintptr) or 0: per view and per OTHER agent b of the
 *                         environment, [0] the pixels of the image won by b's box ("visible") and [1] the
 *                         pixels at which b's box drawn alone (no map, no other agent) leaves a fragment
 *                         within [near, far] ("unoccluded"); 100 * (1 - visible / unoccluded) is the road
 *                         user's occlusion percentage as the renderer sees it (Sec. 5.2, counterfactual
 *                         probes; the paper gives no formula, this is the reading taken).  Entries of the
 *                         ego itself and of inactive agents are 0; the entries of the rendered views are
 *                         overwritten, indexed by absolute view.  Costs an extra pass over the agents' boxes
 *                         and selects the general kernels.
 *   PIC_OPT_OUT_RELATIVE  1: out_class / out_depth (and the PIC_OPT_DEPTH32 image) hold only the rendered
 *                         views, the first rendered view at offset 0 -- so a batch can be streamed in
 *                         passes through buffers of count*H*W pixels (the paper's renderer likewise
 *                         streams a batch in passes bounded by free memory, App. "Renderer memory
 *                         usage"); 0: the images are indexed by absolute view.
 *   PIC_OPT_DEBUG_FLAGS   bit 0: rasterize large primitives without the per-cell trivial
 *                         accept/reject; bit 1: shrink the fused kernel's record pool and the
 *                         cooperative kernel's record list to 2 entries so that the overflow paths
 *                         run; bit 2: send every tile to the cooperative kernel; bit 3: shrink the
 *                         record pool to 40 so that both kernels share the tiles.  All leave the
 *                         images unchanged (tests rely on it); other bits are ignored.
 *   PIC_OPT_TIMING        1: bracket the render kernels of every call with CUDA events on its stream
 *                         (up to 1024 launches between two pic_get_kernel_times calls); 0: off.
 *                         Turning it on creates the events (allocates), so do it outside timed code.
 */
#define PIC_OPT_BRUTE_FORCE 1
#define PIC_OPT_DEPTH32 2
#define PIC_OPT_COUNTERS 3
#define PIC_OPT_VIEW_FIRST 4
#define PIC_OPT_VIEW_COUNT 5
#define PIC_OPT_TIMING 6
#define PIC_OPT_DEBUG_FLAGS 7
#define PIC_OPT_OUT_RELATIVE 8
#define PIC_OPT_OCCLUSION 9
pic_status pic_scene_set_option(pic_scene* scene, int32_t option, uint64_t value);

/*
 * Device time of each render-kernel launch recorded since the last call (PIC_OPT_TIMING on), in
 * milliseconds, oldest first: waits for the last recorded launch, writes min(*n, capacity) values
 * to ms (host) and the number recorded to *n, then forgets them.
 */
pic_status pic_get_kernel_times(pic_scene* scene, float* ms, int32_t capacity, int32_t* n);

/*
 * Host-only: run the scene builder's map preprocessing (pairing of triangles into planar quads,
 * Morton-ordered leaves of up to 8 primitives, groups of 32 leaves) on the maps of `desc` without
 * touching a GPU, and report what it produced.  Only num_maps, map_tri_offset, tri_xyz, tri_class
 * and A of `desc` are read.  out[0..7] = primitives, of which quads, leaves, groups, largest leaf,
 * primitives lying outside their leaf box, leaves lying outside their group box, triangles accounted
 * for (2 per quad + 1 per triangle primitive; equals the input count).  Useful for sizing and
 * for checking the hierarchy's invariants (out[5] == out[6] == 0).
 */
pic_status pic_map_stats(const pic_scene_desc* desc, int64_t out[8]);

/*
 * Colour output: the paper's image format (Sec. 3.2, "I in [0,1]^(h x w x 3)": flat-shaded primitives,
 * cuboids coloured per face with depth-aware brightness, each kind of road user in its own hue,
 * analytic-coverage antialiasing at one sample per pixel).  The paper gives no formulas; this library's are:
 *   colour   pic_set_palette gives every class id an RGB triple (host u8 [256][3]; copied, the call returns
 *            when the copy is done; until it is called class c is the grey (c, c, c)).  A map triangle has its
 *            class's colour; face f of an agent's box has its class's colour times s_f * beta(z),
 *            s = (rear 0.60, front 1.00, right 0.70, left 0.85, bottom 0.40, top 0.92),
 *            beta(z) = 1 - 0.5 (z - near) / (far - near), z the fragment's depth; ground and sky have their
 *            classes' colours.  A channel is stored as floor(c + 0.5), c in [0, 255].
 *   antialias == 0   a pixel shows the primitive that pic_render's class image shows there.
 *   antialias != 0   box filter over the pixel's unit square.  A primitive's coverage of a pixel is the exact
 *            area of the square inside its edges and within [near, far] along its plane; it leaves a fragment
 *            wherever that area is positive, at the depth of its plane at the pixel centre.  A pixel's fragments are
 *            composited front to back; consecutive fragments of one surface -- map triangles of one class, the
 *            faces of one box (only those turned towards the camera are drawn) -- are first merged into one
 *            layer -- nearest first, each adds its coverage, and its colour with that weight, until the layer is
 *            full -- so meshes show no seams and a line thinner than a pixel keeps its share.
 *   out_rgb  dev u8 [E, A, K, H, W, 3].  Arguments, view sub-range options, PIC_OPT_OUT_RELATIVE and
 *            PIC_OPT_TIMING as in pic_render; the other options do not apply.
 * Limits: see PIC_FLAG_COLOUR_INCOMPLETE and PIC_FLAG_COLOUR_FRAGMENTS (reported by pic_get_status, never silently).
 */
pic_status pic_set_palette(pic_scene* scene, const uint8_t* rgb_host, void* cuda_stream);
pic_status pic_render_rgb(pic_scene* scene, const float* poses, const float* dims, const uint8_t* active,
                          const pic_camera* rig_host, int32_t antialias, uint8_t* out_rgb, void* cuda_stream);
/* pic_step with colour output: the bicycle update of pic_step, then pic_render_rgb from the new state. */
pic_status pic_step_rgb(pic_scene* scene, const float* actions, const pic_camera* rig_host, int32_t antialias,
                        uint8_t* out_rgb, void* cuda_stream);

/*
 * pic_render_static -- render without a scene object and without any allocation.
 * (The paper has no counterpart; this entry point exists for callers of this library.)
 *
 * Who needs it: code that is not allowed to obtain device memory at the point where it wants
 * images -- a process whose memory pool was sized and locked at start-up, a real-time loop that
 * must not enter the allocator, a plug-in running under a host application that owns the heap, or
 * a tool that must keep working when the device is nearly full.  pic_scene_create allocates (map
 * copy, hierarchy, per-agent and per-view buffers), so those callers cannot use the scene API.
 *
 * What it does: the same image definition as pic_render, computed by a variant of the exhaustive
 * kernel that reads the caller's triangles directly (one map shared by all environments, every
 * triangle against every pixel -- meant for small batches and small maps).  Per-agent geometry,
 * per-view cameras, per-camera tables and the status word live in one fixed device array that is
 * part of the library image (about 420 KB on every device that loads the library, until exit).
 * The call itself uses no cudaMalloc/cudaFree and no allocating library routine.
 *
 * Limits (PIC_ERR_CAPACITY beyond them): E*A <= PIC_STATIC_MAX_AGENTS, E*A*K <= PIC_STATIC_MAX_VIEWS,
 * H, W <= PIC_STATIC_MAX_SIDE, n_tris <= PIC_STATIC_MAX_TRIS, K <= 16, and, because every primitive
 * is tested against every pixel of every view by one launch that cannot be interrupted,
 * (n_tris + 6*A) * E*A*K*H*W <= PIC_STATIC_MAX_WORK (a few tenths of a second on a B200).
 *
 *   tri_xyz    dev f32 [n_tris,3,3], tri_class dev u8 [n_tris]   (may be NULL when n_tris == 0)
 *   poses, dims, active, rig, out_class, out_depth: as in pic_render (outputs need no alignment)
 * Renders on the CURRENT device, asynchronously on `cuda_stream`.  The first call on a device looks
 * up the array's device address and sets a kernel attribute; make that first call outside any
 * stream capture.  All calls on a device share the one array and it keeps the previous call's
 * contents: the call clears what must start at zero itself, but two calls whose kernels overlap
 * on the GPU (different streams, or several host threads) race on it -- serialise them.
 * A non-finite pose or size makes that agent inactive (its images are sky), as in pic_render, and
 * sets PIC_FLAG_NONFINITE_POSE in a sticky word inside the same array; pic_static_status
 * synchronises `cuda_stream`, copies that word to *flags (host) and clears it -- it allocates
 * nothing either, and reports 0 on a device where pic_render_static has not run yet.
 */
#define PIC_STATIC_MAX_AGENTS 1024
#define PIC_STATIC_MAX_VIEWS 4096
#define PIC_STATIC_MAX_SIDE 512
#define PIC_STATIC_MAX_TRIS 65536
#define PIC_STATIC_MAX_WORK 274877906944.0 /* 2^38 primitive-pixel tests */
typedef struct {
    uint32_t size;                 /* = sizeof(pic_static_desc)                                  */
    int32_t E, A, K, H, W;
    int32_t n_tris;
    float near_z, far_z;
    uint8_t agent_class, sky_class, ground_class, reserved;
} pic_static_desc;
pic_status pic_render_static(const pic_static_desc* desc, const float* tri_xyz, const uint8_t* tri_class,
                             const float* poses, const float* dims, const uint8_t* active, const pic_camera* rig,
                             uint8_t* out_class, uint16_t* out_depth, void* cuda_stream);
pic_status pic_static_status(uint32_t* flags, void* cuda_stream);

/*
 * Measurement aids (the paper has no counterpart): the two microbenchmarks that give a roofline its
 * denominators on the machine at hand.  Both run on the CURRENT device, asynchronously on
 * `cuda_stream`, allocate nothing, and are timed by the caller (CUDA events around the call).
 *   pic_probe_fill   writes `bytes` bytes at dst (dev, 16-byte aligned, bytes % 16 == 0) with 128-bit
 *                    stores from 32 CTAs per multiprocessor: the write-only stream the image store
 *                    competes with.
 *   pic_probe_ffma   runs a register-only loop of `iters` x 8 independent fused multiply-adds per
 *                    thread on 8 CTAs of 256 threads per multiprocessor; out (dev) must hold 2048 floats
 *                    per multiprocessor (out_floats is checked), *fma_count (host) receives the number of
 *                    per-lane multiply-adds the launch executes.
 */
pic_status pic_probe_fill(void* dst, uint64_t bytes, void* cuda_stream);
pic_status pic_probe_ffma(float* out, uint64_t out_floats, int32_t iters, uint64_t* fma_count, void* cuda_stream);

/* Thread-local, never NULL; valid until the next failing call on this thread. */
const char* pic_last_error(void);

/* Library version (major*10000 + minor*100 + patch). */
int32_t pic_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PICTURA_H */
