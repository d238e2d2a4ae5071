/*
 * asymgemm.h - C ABI of the asymmetry-aware persistent BF16 GEMM library for NVIDIA B200
 * (sm_100a).
 *
 * The library follows "Dissecting How Die Scaling Breaks GPU Fine-grained Scheduling":
 * first discover the chip-specific compute topology (Section 5) and the memory-affinity
 * layout (Section 6), then let a persistent kernel use both to decide which physical SMs
 * run and which output tiles each one takes (Section 7.1.2, lessons of Section 7.4.1).
 *
 * Conventions
 *   - Every call returns an ag_status; nothing throws, nothing calls exit().
 *   - "host" / "device" is stated for every pointer.  Device pointers are plain CUDA
 *     device addresses on the current device (cudaSetDevice is the caller's business).
 *   - ag_topo_map and ag_policy are caller-owned plain structs.  ag_affinity_map and
 *     ag_plan are library-owned opaque handles released by the matching *_destroy.
 *   - There is no CPU fallback: on a device that is not compute capability 10.x the
 *     calls that launch kernels return AG_ERR_UNSUPPORTED_ARCH.
 *   - Every device-side wait is bounded; if one runs out the kernel records
 *     AG_ERR_TIMEOUT in the plan's status word (see ag_last_status) and returns.
 *   - A handle (plan, affinity map, packed weights, group descriptor) may be used by one host
 *     thread at a time; launches of one plan must not overlap on the device (use one plan per
 *     stream).  Different plans may run concurrently on disjoint SM sets (avoid_sm_mask).
 *   - gemm_persistent, gemm_persistent_packed, gemm_persistent_grouped, gemm_persistent_noalloc and
 *     attention_decode_persistent return AG_ERR_ARG, and queue nothing, when cuda_stream is being captured: every launch carries
 *     a launch number (epoch) in its kernel parameters, by which the thread blocks take their places
 *     in the plan; a replayed graph would repeat an old number and no block would join.
 *   - Environment: AG_DEBUG=1 makes topo_discover print its bandwidth measurements and any
 *     rejected latency rows to stderr.  Nothing else is read from the environment.
 */
#ifndef ASYMGEMM_H_
#define ASYMGEMM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AG_MAX_SM 256
#define AG_MAX_GPC 32
#define AG_MAX_DIE 2
#define AG_CHUNK_BYTES 4096 /* partition interleave granularity reported in Section 6.1.2 */

typedef enum {
    AG_OK = 0,
    AG_ERR_ARG = 1,              /* null pointer, bad size, misaligned buffer, plan/shape mismatch */
    AG_ERR_CUDA = 2,             /* a CUDA runtime/driver call failed (see ag_last_cuda_error) */
    AG_ERR_UNSUPPORTED_ARCH = 3, /* device is not sm_100 */
    AG_ERR_TIMEOUT = 4,          /* a bounded device-side wait ran out */
    AG_ERR_UNMANNED_SM = 5,      /* an SM of the plan never got a thread block */
    AG_ERR_NOISY_PROBE = 6,      /* latency tiers could not be separated */
    AG_ERR_STALE_AMAP = 7,       /* affinity map does not belong to this buffer */
    AG_ERR_NOMEM = 8
} ag_status;

/* ---- compute topology (Section 5, Section 6.1.1) -------------------------------------- */
typedef struct {
    int32_t n_sm, n_tpc, n_gpc, n_die;
    int32_t tpc[AG_MAX_SM];        /* TPC of SM s: two consecutive SM ids share a TPC (Section 5.1.2) */
    int32_t gpc[AG_MAX_SM];        /* GPC class of SM s, -1 if it could not be placed */
    int32_t die[AG_MAX_SM];        /* memory-affinity partition (die) of SM s; die 0 = die of SM 0 */
    uint8_t is_random[AG_MAX_SM];  /* 1: never seen in a thread-block cluster larger than 2 (Section 5.1.1) */
    int32_t die_sm_count[AG_MAX_DIE];
    int32_t gpc_sm_count[AG_MAX_GPC];
    int32_t gpc_die[AG_MAX_GPC];
    uint32_t lat_near_cycles, lat_far_cycles, lat_threshold; /* HBM latency tiers seen by the probe */
    uint32_t l2_near_cycles, l2_far_cycles;                  /* L2-hit latency, same-die / other-die reader */
    int32_t n_unplaced;            /* SMs left with gpc == -1 */
    int32_t device;                /* CUDA device ordinal the map was measured on */
    uint32_t sm_clock_khz;         /* SM clock rate reported by the device at probe time */
    uint32_t flags;                /* AG_TOPO_* bits of the phases that ran */
} ag_topo_map;

#define AG_TOPO_CENSUS 1u
#define AG_TOPO_CLUSTER 2u
#define AG_TOPO_LATENCY 4u
#define AG_TOPO_BANDWIDTH 8u

/*
 * topo_discover - build the SM -> TPC/GPC/die map of the current device.
 * Section 5.1.1 (cluster probing: SMs that co-occur in a thread-block cluster share a GPC),
 * Section 5.1.2 (L2-bandwidth probing places the remaining "random" SMs),
 * Section 6.1.1 (HBM latency seen from every SM splits the SMs into two partitions).
 *   map  host pointer, caller-owned, fully overwritten.
 * Allocates and frees its own device scratch; synchronises the device.
 * Errors: AG_ERR_ARG (null), AG_ERR_UNSUPPORTED_ARCH, AG_ERR_CUDA, AG_ERR_NOISY_PROBE
 * (two latency tiers not found), AG_ERR_UNMANNED_SM (census did not see every SM).
 */
ag_status topo_discover(ag_topo_map* map);

/* Same with a choice of phases (AG_TOPO_* bits); skipped phases leave gpc = -1 / die = 0. */
ag_status ag_topo_discover_phases(ag_topo_map* map, uint32_t phases);

/*
 * ag_topo_from_observations - the host half of topo_discover on recorded observations
 * (no device needed): union-find over cluster co-occurrence (Section 5.1.1) and two-tier
 * split of per-SM latency vectors (Section 6.1.1).
 *   cluster_sm[cluster_off[c] .. cluster_off[c+1])  SM ids seen together in cluster c (host)
 *   lat[s * n_ref + r]  min latency in cycles from SM s to reference chunk r (host)
 *   map  host, out.  Errors: AG_ERR_ARG, AG_ERR_NOISY_PROBE.
 */
ag_status ag_topo_from_observations(int32_t n_sm, const int32_t* cluster_sm, const int32_t* cluster_off,
                                    int32_t n_clusters, const uint32_t* lat, int32_t n_ref,
                                    ag_topo_map* map);

/*
 * ag_topo_place_by_gain - decision rule of Section 5.1.2 for one unplaced TPC: given the
 * bandwidth gain (bytes/s) of adding the TPC to the known SMs of each candidate GPC and the
 * TPC's solo bandwidth, return the index of the GPC it contends with (smallest gain, below
 * solo_bw * margin while the runner-up is above it), or -1 if the sweep is ambiguous.
 */
int32_t ag_topo_place_by_gain(const double* gain, int32_t n_candidates, double solo_bw);

/* Keep a map in a file / read it back (the paper budgets up to a minute per GPU for discovery,
 * Section 5.1.2).  Loading checks the file's magic, size and internal consistency; a map belongs
 * to the GPU it was measured on (map->device).  Errors: AG_ERR_ARG. */
ag_status ag_topo_save(const ag_topo_map* map, const char* path);
ag_status ag_topo_load(const char* path, ag_topo_map* map);

/*
 * ag_probe_latency_samples - raw access-latency samples from one SM: the measurement behind the
 * HBM and L2 latency histograms of Section 6.1.1 (kernels in the appendix).  Line r lies in
 * 4 KB chunk (29 r + 3) mod 2048 of a library-owned 8 MiB scratch buffer.
 *   sm     SM id that takes the samples
 *   mode   0: invalidate the L2 line before each timed load (HBM latency);
 *          1: plain timed L1-bypassing load (latency of whichever level holds the line)
 *   cycles host, out, n_lines x reps values (n_lines <= 1024, reps <= 64), SM clock cycles
 * Errors: AG_ERR_ARG, AG_ERR_UNSUPPORTED_ARCH, AG_ERR_CUDA, AG_ERR_UNMANNED_SM.
 */
ag_status ag_probe_latency_samples(int sm, int mode, int n_lines, int reps, uint32_t* cycles);

/*
 * ag_probe_l2_bandwidth - aggregate L2 read bandwidth (bytes/s) of a chosen set of SMs, the
 * measurement behind Section 5.1.2 (and its per-GPC bandwidth figure): every SM of the set
 * re-reads a 1 MiB slice (larger than L1, all slices together far smaller than L2) with
 * L1-bypassing loads; best of three runs.
 *   sm_mask  host, bit s = SM s takes part.  bytes_per_s  host, out.
 * Errors: AG_ERR_ARG, AG_ERR_UNSUPPORTED_ARCH, AG_ERR_CUDA, AG_ERR_UNMANNED_SM.
 */
ag_status ag_probe_l2_bandwidth(const uint64_t sm_mask[4], double* bytes_per_s);

/* ---- memory affinity (Section 6.1) ------------------------------------------------------ */
typedef struct ag_affinity_map ag_affinity_map;

/*
 * affinity_probe - chunk -> die map of a device buffer from access latency (Section 6.1.1 and
 * the latency kernels of the appendix: a single thread invalidates the L2 line, loads it with an
 * L1-bypassing load and times the round trip with the SM cycle counter; the minimum over several
 * lines and repeats of the chunk is kept).  Every chunk is timed from the SMs of die 0 and from
 * the SMs of die 1; it belongs to the die that reaches it faster.  A chunk is AG_CHUNK_BYTES;
 * die 0 is the die of SM 0.
 *   buf    device pointer, 4096-byte aligned; contents are preserved (each probed 128-byte
 *          line is saved before the L2 invalidation and written back afterwards).  Nothing
 *          else may touch the buffer while the probe runs.
 *   bytes  multiple of 4096.
 *   amap   host, out: new handle.
 * affinity_probe runs the census + latency phases of topo_discover itself;
 * ag_affinity_probe_with_map takes a map that already has them.  Synchronises the device.
 * Errors: AG_ERR_ARG, AG_ERR_UNSUPPORTED_ARCH, AG_ERR_CUDA, AG_ERR_NOISY_PROBE (more than 2 % of
 * the chunks show no clear difference between the dies), AG_ERR_UNMANNED_SM, AG_ERR_NOMEM.
 */
ag_status affinity_probe(void* buf, size_t bytes, ag_affinity_map** amap);
ag_status ag_affinity_probe_with_map(void* buf, size_t bytes, const ag_topo_map* map,
                                     ag_affinity_map** amap);
/* Build a handle from a given chunk->die table (host, one byte per chunk, values 0/1):
 * lets plans be built for a recorded or synthetic layout. */
ag_status ag_affinity_from_table(const void* buf, size_t bytes, const uint8_t* die_of_chunk,
                                 size_t n_chunks, ag_affinity_map** amap);
/* Copy out the chunk->die table (host, cap bytes). */
ag_status ag_affinity_export(const ag_affinity_map* amap, uint8_t* die_of_chunk, size_t cap,
                             size_t* n_chunks);
/* Raw min-latency cycles (host, cap >= 2 * n_chunks words): first the values seen from die 0,
 * then those seen from die 1.  Only for probed maps. */
ag_status ag_affinity_cycles(const ag_affinity_map* amap, uint32_t* cycles, size_t cap);
/* Section 6.1.1: the two groups of SMs see opposite tiers.  *mismatches = number of chunks whose
 * two latencies were less than 25 % apart, i.e. that did not show opposite tiers. */
ag_status ag_affinity_check_complement(const ag_affinity_map* amap, const ag_topo_map* map,
                                       size_t* mismatches);
/*
 * ag_affinity_fit_hash - partition-hash recovery (Section 6.1.2) from a measured map: which of the
 * nine chunk-index bits inside a 2 MiB page (address bits 12..20) take part in the XOR (parity)
 * hash.  Bit b of *mask is set when flipping chunk-index bit b changes the die of most chunks.
 * *violations (host, may be NULL) = chunks whose die is not parity(index-in-page & mask) ^ c for
 * the best per-page constant c (measurement noise, or a layout that is not such a hash).  Address
 * bits above 20 are not visible without physical addresses; they end up in the per-page constants.
 * Needs a map of at least 4 MiB.  Errors: AG_ERR_ARG.
 */
ag_status ag_affinity_fit_hash(const ag_affinity_map* amap, uint32_t* mask, size_t* violations);
/*
 * ag_probe_die_bandwidth - local against remote memory bandwidth (Section 6.2.1: the 4 KB pages of a
 * region are classified by partition and a read kernel is restricted to the local or the remote ones).
 * The SMs of reader_die stream all chunks of the mapped buffer that belong to chunk_die (at least 1 GiB in
 * total, several passes if needed; use a buffer well above the L2 size to measure HBM rather than L2).
 *   bytes_per_s  host, out: best of three runs.
 * Reads only; the buffer must be the one the map was probed on.  Synchronises the device.
 * Errors: AG_ERR_ARG, AG_ERR_UNSUPPORTED_ARCH, AG_ERR_CUDA, AG_ERR_UNMANNED_SM.
 */
ag_status ag_probe_die_bandwidth(const ag_affinity_map* amap, const ag_topo_map* map, int reader_die,
                                 int chunk_die, double* bytes_per_s);
/*
 * ag_probe_ring_bandwidth - what a ring of shared-memory stages filled by bulk copies reads from memory: the copy side of
 * the streaming kernels (decode-shaped GEMM, attention decode) without their arithmetic, to choose policy.ring_stages
 * for a chip.  n_blocks blocks (one per SM: each takes 200 KB of shared memory) stream equal contiguous shares of buf;
 * each keeps `stages` buffers of `stage_bytes` in flight, refilled by `producers` warps in turn; one thread takes the
 * stages off in order, spends hold_ns on each (one after the other, as a thread that issues a stage's MMAs does; 0 = none)
 * and hands it back.
 *   buf    device, 16-byte aligned, read only; bytes >= n_blocks * stage_bytes (use far more than the L2 size)
 *   stages 1..8, stage_bytes a multiple of 4096 in 4096..65536, stages * stage_bytes <= 192 KiB
 *   producers 1..3 and <= stages; hold_ns 0..100000
 *   bytes_per_s  host, out: best of three runs (first block's start to last block's end).
 * Synchronises the device.  Errors: AG_ERR_ARG, AG_ERR_UNSUPPORTED_ARCH, AG_ERR_CUDA, AG_ERR_TIMEOUT (a bounded wait
 * ran out; the device stays usable).
 */
ag_status ag_probe_ring_bandwidth(const void* buf, size_t bytes, int n_blocks, int stages, int stage_bytes,
                                  int producers, int hold_ns, double* bytes_per_s);
void ag_affinity_destroy(ag_affinity_map* amap);

/* ---- plan (Section 7.1.2) ------------------------------------------------------------ */
enum { AG_OBLIVIOUS = 0, AG_DIE_COMPACT = 1, AG_AFFINITY = 2 };
enum { AG_LAYOUT_ROWMAJOR = 0, AG_LAYOUT_PAGED = 1 };

typedef struct {
    int32_t present;        /* 0: operand not counted by the affinity policy */
    int32_t layout;         /* AG_LAYOUT_ROWMAJOR: rows of row_stride bytes; AG_LAYOUT_PAGED: B only, 4 KB pages of
                               [128 columns x 16 k] elements, page of (pc, k16) = pc*ceil(K/16)+k16 with pc the index
                               of the 128-column block (a unit column of width tile_n holds tile_n/128 blocks) */
    int64_t offset;         /* byte offset of element (0,0) from the probed buffer's base */
    int64_t row_stride;     /* bytes between rows (row-major) */
    int32_t elem_bytes;
    int32_t reserved;
    const int32_t* page_table; /* host; AG_LAYOUT_PAGED: chunk index (in the probed buffer) of each logical page */
    int64_t n_pages;
} ag_operand_desc;

typedef struct {
    int32_t kind;            /* AG_OBLIVIOUS | AG_DIE_COMPACT | AG_AFFINITY */
    int32_t M, N, K;
    int32_t tile_m, tile_n;  /* dense kernel: 128 x {64,128,256}, or 256 x 256 (two thread blocks on the two SMs of a TPC
                                share a unit; the plan's SM set must consist of whole TPCs, else AG_ERR_ARG);
                                decode-shaped kernel: {16,32,64} x 128, and 128 x 128 with decode_shaped = 1 */
    int32_t k_splits;        /* >= 1, runs of whole k-slabs (no run may be empty).  Decode-shaped plans: few, large units stream
                                best - measured at N = K = 8192 on 148 SMs: 4 splits (256 units of 512 KB of weights) reach the
                                memory's limit, 16 splits 0.9 of it; on a partial chip take enough splits for about 7 units per
                                SM, so that the longest list is not much longer than the average */
    int32_t k_unit;          /* elements per k-slab (64) */
    int32_t raster_group;    /* tile rows per raster group (>= 1) */
    int32_t preferred_die;   /* -1: the die with more usable SMs */
    int32_t invert_affinity; /* 1: send every unit to the die that holds fewer of its bytes */
    int32_t static_assign;   /* 1: static per-SM lists (the paper's mode); 0: CTAs pull from per-die queues */
    uint64_t seed;           /* oblivious only: 0 = lowest SM ids, else seeded random subset */
    int64_t min_margin;      /* affinity only: byte margins below this count as ties (0 = exact ties only) */
    int32_t splitk_in_memory; /* decode-shaped plans with k_splits > 1: 0 = partial sums go through a
                                 workspace and are added in ascending split order by a small second kernel
                                 launched behind the GEMM (bit-reproducible);
                                 1 = C is zeroed and every unit adds its partial sums with reductions in
                                 memory (no workspace, no waiting; the order of the fp32 adds is not fixed) */
    int32_t sm_select;       /* die_compact / affinity: 0 = primary die first (die-compact set); 1 = whole TPCs dealt
                                round-robin over the GPCs of both dies (fewest SMs per GPC, Section 5.1.2) */
    int32_t pair_lists;      /* 1: static lists are dealt to TPCs instead of SMs (entry i of a die's queue -> TPC i mod P,
                                lower SM in even rounds, upper SM in odd ones), so that the two lists of a TPC together
                                hold a fair share; for plans of block pairs.  Needs whole TPCs, else AG_ERR_ARG */
    int32_t overlap_launches; /* decode-shaped plans with static lists (ignored otherwise): 1 or 2 =
                                 a launch lets the next launch of this library on the same stream begin while it is still
                                 finishing (programmatic dependent launch): the next launch's thread blocks take over SMs as
                                 they become free and start streaming their weights (attention: key/value pages); nothing
                                 of theirs is written before this launch has completed.  The caller promises that the
                                 weights (B / packed weights, KV pages) of a call are not produced by the call directly
                                 before it.  1: the activations (A, queries) may be - they are read only after the launch
                                 before has completed; 2: the caller promises the same for the activations, and they are
                                 read at once.  0 = launches run strictly one after the other.  On a plan for part of
                                 the chip the next launch's surplus blocks wait on the unplanned SMs until the running
                                 launch has left the planned ones: use it when the stream has the chip to itself, not
                                 while another stream's kernels are meant to run on the unplanned SMs */
    int32_t cluster_size;    /* die_compact / affinity: thread-block cluster size (1, 2, 4 or 8) of the kernel the SM set is
                                meant for; 0 and 1 mean none.  For sizes above 2 the set is built from what can host such
                                clusters: SMs never seen in a cluster larger than 2 (is_random, Section 5.1.1) are taken last,
                                and every GPC contributes whole blocks of cluster_size normal SMs - a GPC hosts only
                                floor(n / cluster_size) clusters on n SMs (Section 7.3: twelve SMs form three clusters of
                                four but one cluster of eight).  ag_cluster_capacity counts what a set can host */
    int32_t die_quota;       /* die_compact / affinity: how the units are shared between the dies.  0 = in proportion to the
                                SMs the set has on each die (right for work that is bound by the SMs).  1 = equal shares for
                                the dies that hold any SM of the set: for work bound by memory bandwidth whose operands are
                                die-local, since every die's memory delivers the same bandwidth whatever its SM count (on a
                                chip with 70 and 78 usable SMs the proportional split asks 5 % more of one die's memory) */
    int32_t decode_shaped;   /* 1: a plan with tile_m = 128 and tile_n = 128 is run by the decode-shaped (weight-streaming)
                                kernel - weights on the MMA's M side, up to 128 activation rows on its N side - instead of
                                the dense one-block kernel.  Plans with tile_m <= 64 (and tile_n = 128) always are */
    int32_t ring_stages;     /* decode-shaped GEMM and attention decode: stages of 32 KB that a block keeps in flight from
                                memory (2..6, clamped to what the kernel has; even for up to 32 activation rows).  0 =
                                default: attention decode shares 20 MiB between the plan's SMs (4 stages on the full
                                chip, where more in flight oversubscribes the memory system; 6 on half of it), the
                                decode-shaped GEMM uses all its stages, except four for units of at most 128 KB of
                                row-major weights or of pages in consecutive chunks */
    uint64_t avoid_sm_mask[4]; /* bit s set: SM s belongs to another plan */
    ag_operand_desc a, b, c;
} ag_policy;

typedef struct ag_plan ag_plan;

/*
 * sched_build - choose sm_budget physical SMs and give every work unit (output tile x
 * k-split) to exactly one of them.  Section 7.1.2: persistent block per SM, schedule planned
 * in advance, each block takes the tasks whose data lives in its SM's partition, work split
 * between partitions in proportion to their SM counts; static assignment (Section 7.4.1).
 * The plan is computed by CUDA kernels and stays on the device for gemm_persistent.
 *   map     host, from topo_discover (or any consistent map with n_sm = device SM count)
 *   amap    handle or NULL; required for AG_AFFINITY
 *   policy  host
 *   plan    host, out: new handle
 * At most 2^20 work units, whatever the policy (the affinity policy finds each die's share with a radix
 * select over the units' byte margins, not a sort).
 * Errors: AG_ERR_ARG (budget out of range, bad tile shape, empty k-split, more than 2^20 units, operand
 * outside the probed buffer, AG_AFFINITY without amap), AG_ERR_CUDA, AG_ERR_NOMEM.
 */
ag_status sched_build(const ag_topo_map* map, const ag_affinity_map* amap, int sm_budget,
                      const ag_policy* policy, ag_plan** plan);
/* Flat int32 image of the plan (host, cap words): header[16] = magic 0x41475031, kind, n_sm,
 * b, n_die, n_units, tiles_m, tiles_n, k_splits, tile_m, tile_n, M, N, K, static_assign, 0;
 * then sm_list[b], sm_die[b], rank_in_die[b], die_sm_count[2], die_q_off[3], die_q[n_units],
 * sm_q_off[b+1], sm_q[n_units], smid_to_slot[n_sm]. */
ag_status ag_plan_export(const ag_plan* plan, int32_t* out, size_t cap, size_t* n_words);
/* Affinity margins local_0 - local_1 per raster index (host, cap entries), for spot checks. */
ag_status ag_plan_margins(const ag_plan* plan, int64_t* out, size_t cap);
/* Executed-by record of the last launches: SM id that ran unit u and how often it ran
 * (host arrays of n_units entries, either may be NULL); ag_plan_reset_record zeroes the counts. */
ag_status ag_plan_tile_record(const ag_plan* plan, int32_t* owner_sm, int32_t* run_count, size_t cap);
ag_status ag_plan_reset_record(ag_plan* plan);
/*
 * ag_plan_trace / ag_plan_unit_times - per-unit timeline of the last launch, for load-balance and tail
 * analysis (the paper profiles its kernels with hardware counters; this is the software counterpart).
 * With tracing on, every kernel stamps the global nanosecond timer when a unit is handed to the block's
 * pipeline (start) and when its last output has been issued (end); unit u's pair is returned in
 * start_ns[u], end_ns[u] (host, cap >= n_units; 0 = the unit did not run).  Cost: two 8-byte stores per unit.
 * Errors: AG_ERR_ARG (tracing off, small cap), AG_ERR_CUDA, AG_ERR_NOMEM.
 */
ag_status ag_plan_trace(ag_plan* plan, int on);
ag_status ag_plan_unit_times(const ag_plan* plan, uint64_t* start_ns, uint64_t* end_ns, size_t cap);
/*
 * ag_plan_set_grid - launch fewer thread blocks than the device has SMs (blocks = 0 restores one
 * block per SM), e.g. when part of the GPU is known to be busy.  Planned SMs that get no block are
 * then "unmanned": with static lists, a block that has finished its own list takes over the list
 * of an unmanned SM (Section 7.1.2 plans per SM; the take-over keeps the plan complete), with
 * dynamic queues the per-die queues are simply drained by fewer blocks.  Not available for plans of
 * block pairs (tile_m = 256).  ag_plan_adopted reports how many lists have been taken over since the
 * plan was built.  Errors: AG_ERR_ARG.
 */
ag_status ag_plan_set_grid(ag_plan* plan, int blocks);
ag_status ag_plan_adopted(const ag_plan* plan, uint32_t* n_lists);
/* Thread-block clusters of cluster_size blocks that the plan's SM set can host at once with one block per SM: per GPC
 * floor(normal SMs of the set in that GPC / cluster_size); SMs with is_random set or without a GPC host none when
 * cluster_size > 2 (Sections 5.1.1, 7.3).  Errors: AG_ERR_ARG. */
ag_status ag_cluster_capacity(const ag_plan* plan, const ag_topo_map* map, int cluster_size, int32_t* n_clusters);
/*
 * ag_probe_cluster_layout - where the hardware puts thread-block clusters (Section 5.1.1 probes the same way): launches
 * n_clusters clusters of cluster_size blocks (one block per SM, every block stays until all have started or 50 us have
 * passed) and reports, per SM id, the cluster that ran there first (-1: none).
 *   cluster_of_sm  host, out, AG_MAX_SM entries
 * Errors: AG_ERR_ARG (size not in 2..8, n_clusters < 1), AG_ERR_UNSUPPORTED_ARCH, AG_ERR_CUDA.
 */
ag_status ag_probe_cluster_layout(int cluster_size, int n_clusters, int32_t* cluster_of_sm);
/* Device status word of the most recent launch (call after synchronising its stream). */
ag_status ag_last_status(const ag_plan* plan);
/* Where the first bounded wait of the last launches ran out (only meaningful while ag_last_status is AG_ERR_TIMEOUT):
 * role = which wait of which warp role gave up (1-2 scheduler and copy warps waiting for room, 3-5 the MMA issuer
 * waiting for a unit / an accumulator / data, 6-7 the epilogue or softmax warps, 8-9 copy warps and the MMA issuer
 * waiting for a unit or activations), smid = the SM it happened on; 0 and -1 when nothing ran out.  Either may be NULL. */
ag_status ag_last_status_where(const ag_plan* plan, int32_t* role, int32_t* smid);
void ag_plan_destroy(ag_plan* plan);

/*
 * gemm_persistent - C = A * B on the SMs of the plan.  One persistent thread block per
 * planned SM reads %smid, takes its slot of the plan and loops over its work units
 * (Section 7.1.2); TMA feeds shared memory, tcgen05 MMAs accumulate in tensor memory in fp32.
 *   A  device, M x K bf16 row-major, 16-byte aligned, K % 8 == 0
 *   B  device, K x N bf16 row-major, 16-byte aligned, N % 8 == 0
 *   C  device, M x N fp32 row-major, 16-byte aligned; overwritten.  Dense plans with k_splits > 1:
 *      zeroed first, partial sums are then added with reductions in memory.  Decode-shaped plans
 *      (see below): see policy.splitk_in_memory
 *   the plan's tile shape selects the kernel: 256 x 256 units = pairs of thread blocks, 128 x
 *      {64,128,256} = one block per tile (any SM set), {16,32,64} x 128 (and 128 x 128 with policy.decode_shaped)
 *      = decode-shaped (M <= tile_m): the weight tile sits on the MMA's M side and is streamed once
 *   plan  built for the same M, N, K, else AG_ERR_ARG
 *   cuda_stream  a cudaStream_t (NULL = default stream).  Asynchronous.
 * Errors: AG_ERR_ARG, AG_ERR_UNSUPPORTED_ARCH, AG_ERR_CUDA.  Device-side trouble
 * (AG_ERR_TIMEOUT, AG_ERR_UNMANNED_SM) is reported by ag_last_status.
 */
ag_status gemm_persistent(const void* A, const void* B, void* C, int M, int N, int K,
                          const ag_plan* plan, void* cuda_stream);

/* ---- die-local packed weights for decode-shaped GEMMs (Section 7.1.1) ------------------------ */
typedef struct ag_packed_weights ag_packed_weights;

/*
 * ag_pack_weights - indirect allocation by remapping (Section 7.1.1 and the remapping appendix,
 * Eq. 1): copy the K x N weights into 4 KB pages of [128 columns x 16 k] elements and store
 * every page in a chunk of the die that the plan gave the page's work unit to.  The destination
 * is read as aligned chunk pairs; two logical views (one per die) are laid over it and page p of
 * view d is the chunk of pair p that the affinity map places on die d (the measured bit stands in
 * for the parity-of-masked-physical-address selector of Eq. 1).  Inside a page element (n, k) sits
 * at byte (n/8)*256 + (k/8)*128 + (n%8)*16 + (k%8)*2, the order the MMA reads without swizzle.
 *   B      device, K x N bf16 row-major
 *   plan   a decode-shaped plan (tile_n = 128, one tile row) or a dense plan with 256-column units
 *          (tile_n = 256: two pages side by side per unit column); K % 64 == 0.  A page read by
 *          units of both dies goes to the die that runs most of them (tie: die 0)
 *   amap   affinity map of exactly (dst, dst_bytes), else AG_ERR_STALE_AMAP
 *   dst    device, 4096-aligned; needs 2 * max(pages of die 0, pages of die 1) chunks
 *   out    host, out: handle holding the page table (device + host copy)
 * Synchronises the device.  Errors: AG_ERR_ARG, AG_ERR_STALE_AMAP, AG_ERR_CUDA, AG_ERR_NOMEM.
 */
ag_status ag_pack_weights(const void* B, int K, int N, const ag_plan* plan, const ag_affinity_map* amap,
                          void* dst, size_t dst_bytes, ag_packed_weights** out);
/*
 * ag_pack_weights_ex - ag_pack_weights / ag_pack_weights_grouped with options (G = 1: B_list holds one matrix).
 *   flags  bit 0: keep the one-page-per-copy layout even where groups of four pages are possible.
 *          bit 1: always read the page tables in the kernel (do not use the closed form below).
 *          bit 2: ignore the dies - logical page p goes to chunk p of dst (the hardware's interleaved placement; dst needs
 *                 one chunk per page).  The page layout stays, a work unit's pages are one contiguous run, and the
 *                 decode-shaped kernel fetches a stage with one plain copy.  The comparison arm for the die-local
 *                 layout, and on the full chip the fastest way to stream the weights.
 * Closed form (Eq. 1 of the remapping appendix, page_phys = 2j + [parity((page_start + 2j) & MASK) xor P]): when the
 * measured map is an exact XOR hash over the chunks in use - in-page mask from ag_affinity_fit_hash, one further bit
 * per 2 MiB page, no chunk out of line - and the plan is decode-shaped, the pages of a work unit are consecutive in
 * the view of its die and the chunk of every page (or the base of every group of four) follows from the unit's first
 * position, the mask and the page bits.  ag_pack_weights recomputes every table entry that way; if all agree, the
 * decode-shaped kernel computes page addresses instead of loading them (one word per unit and one bit per 2 MiB
 * instead of one word per page or group).  Otherwise the tables stay in use.  ag_packed_closed_form reports which.
 * Grouped pages: when the map follows an XOR hash (ag_affinity_fit_hash) that uses chunk-index bits 0 and 1
 * and leaves some bit f in 2..8 out, the chunks {q, q+a, q+F, q+F+a} (F = 2^f; a = 3 for q = 0 mod 4, a = 1
 * for q = 1 mod 4; bit f of q clear) always sit on one die.  The four pages of a k-slab (of one 128-column block)
 * are then stored in one such group and fetched with a single strided copy; groups whose measured
 * chunks disagree are skipped.  ag_packed_info reports f (-1: single pages).
 */
ag_status ag_pack_weights_ex(const void* const* B_list, int G, int K, int N_expert, const ag_plan* plan,
                             const ag_affinity_map* amap, void* dst, size_t dst_bytes, uint32_t flags,
                             ag_packed_weights** out);
ag_status ag_packed_info(const ag_packed_weights* w, int32_t* group_free_bit);
/* *enabled = 1 when the kernels compute page addresses from the fitted hash; mask = the in-page mask; table_bytes /
 * closed_bytes = device bytes of the lookup tables and of the closed form's data (any of the last three may be NULL). */
ag_status ag_packed_closed_form(const ag_packed_weights* w, int32_t* enabled, uint32_t* mask, size_t* table_bytes,
                                size_t* closed_bytes);
/* Page table (host, cap entries): chunk index in dst of logical page (pc, k16) = pc * (K/16) + k16, pc = index
 * of the 128-column block; feed it to ag_operand_desc.page_table to build an affinity plan over the packed weights. */
ag_status ag_packed_page_table(const ag_packed_weights* w, int32_t* out, size_t cap, size_t* n_pages);
void ag_packed_destroy(ag_packed_weights* w);

/*
 * gemm_persistent_packed - C = A * B with the B operand taken from a packed buffer
 * (Section 7.1.2 on top of Section 7.1.1: each block reads the pages of its units, which the
 * packing put on the block's own die when plan and packing agree).  Decode-shaped plans
 * (tile_m in {16, 32, 64, 128}, tile_n = 128, M <= tile_m) and dense plans of block pairs (256 x 256
 * units, SM set of whole TPCs) are accepted; gemm_persistent handles the same shapes with
 * row-major B.
 *   A  device, M x K bf16 row-major, 16-byte aligned;  C  device, M x N fp32 row-major, overwritten
 *   plan  same N, K (and tile_n) as the packing; decode-shaped plans: with
 *         k_splits > 1 the partial sums either go through the plan's workspace and are added in
 *         ascending split order by a second kernel launched behind the GEMM, or are added straight
 *         into a zeroed C by reductions in memory (policy.splitk_in_memory)
 * Asynchronous on cuda_stream.  Errors as gemm_persistent.
 */
ag_status gemm_persistent_packed(const void* A, const ag_packed_weights* W, void* C, int M, int N, int K,
                                 const ag_plan* plan, void* cuda_stream);

/* ---- grouped (MoE-shaped) decode GEMM --------------------------------------------------------
 * The paper's best full-GPU result is a grouped GEMM (Section 7.1.2 and its workload appendix: G
 * experts, expert g multiplies its M_g routed rows by its own K x N weights).  Built here for the
 * decode-shaped case (M_g <= 32): the plan sees the experts side by side as one problem with
 * N = G * N_expert columns, so the die-compact rule gives each die a run of experts, and
 * ag_pack_weights_grouped puts every expert's weights on the die that runs it.
 */
typedef struct ag_group_desc ag_group_desc;
/*
 *   A_all  device, stacked activations: sum(rows) x K bf16 row-major, expert g owns rows
 *          [sum(rows[0..g)), + rows[g])
 *   C_all  device, stacked outputs: sum(rows) x N_expert fp32 row-major, same row ranges
 *   rows   host [G]; decode-shaped descriptors: 0 <= rows[g] <= tile_m; dense descriptors
 *          (tile_m = 256, block pairs, N_expert % 256 == 0): any row count
 *   B_list host array of G device pointers (K x N_expert bf16 row-major each), or NULL when only
 *          packed weights will be used
 *   N_expert % 128 == 0, K % 8 == 0, tile_m in {16, 32, 64, 128, 256}
 * Errors: AG_ERR_ARG, AG_ERR_CUDA, AG_ERR_NOMEM.
 */
ag_status ag_group_desc_create(const void* A_all, void* C_all, const int32_t* rows, int G,
                               const void* const* B_list, int N_expert, int K, int tile_m,
                               ag_group_desc** out);
void ag_group_desc_destroy(ag_group_desc* d);
/* As ag_pack_weights for G weight matrices; plan: N = G * N_expert, tile_n = 128, one tile row. */
ag_status ag_pack_weights_grouped(const void* const* B_list, int G, int K, int N_expert, const ag_plan* plan,
                                  const ag_affinity_map* amap, void* dst, size_t dst_bytes,
                                  ag_packed_weights** out);
/*
 * gemm_persistent_grouped - C_g = A_g * B_g for all experts in one persistent launch.
 *   W     packed weights from ag_pack_weights_grouped, or NULL to read the row-major B_list
 *   plan  M = max rows of an expert, N = G * N_expert, K; decode-shaped: tile_n = 128, M <= tile_m;
 *         dense: tile_m = tile_n = 256, SM set of whole TPCs (units below an expert's last row are
 *         skipped, so prefer static lists built from balanced row counts)
 *   Decode-shaped: a unit of an expert with rows[g] == 0 is ticked off by the scheduling warp without
 *   reading a weight byte (its tile record shows one execution, its C rows do not exist).  Static lists
 *   are cut before the row counts are known; when most experts are idle, dynamic queues
 *   (policy.static_assign = 0) or two k-splits balance the active units better.
 * Asynchronous on cuda_stream; split-K modes as gemm_persistent_packed.  Errors as gemm_persistent.
 */
ag_status gemm_persistent_grouped(const ag_group_desc* d, const ag_packed_weights* W, const ag_plan* plan,
                                  void* cuda_stream);

/*
 * gemm_persistent_noalloc - the decode-shaped gemm_persistent (M <= 32, row-major B) for callers
 * that cannot allocate device memory when they need the result.  (The paper has no counterpart;
 * this entry point exists for deployment reasons only.)
 *
 * Who needs it: a serving process whose own memory pool already owns all of the GPU's free memory,
 * so that cudaMalloc fails; a latency-bound request loop where an allocator call is not
 * acceptable; code that runs after a framework has declared "no more allocations".  The split-K
 * partial sums, which normally live in memory that sched_build attached to
 * the plan, are placed instead in a fixed workspace that is part of the library image: 8 MiB +
 * 16 KiB of device memory per GPU.  The CUDA runtime loads the library's device code onto a GPU
 * when it is first used there, so the workspace (and the kernel itself) takes its memory during
 * the first gemm_persistent_noalloc call on that GPU and keeps it until the process exits.  Make
 * that first call at start-up, while memory is still available (any small problem will do); it can
 * fail with AG_ERR_NOMEM if the GPU is already full.  From the second call on, a call performs no
 * cudaMalloc, cudaFree or other allocating call and leaves the free device memory unchanged.
 *
 * Limits: k_splits * M * N * 4 bytes <= 8 MiB (for example M = 16, N = 8192, k_splits = 16) and
 * N <= 131072; larger problems are refused with AG_ERR_ARG, as are plans that are not
 * decode-shaped with at most 32 rows (tile_m > 32).  Arguments are those of gemm_persistent; the plan may come from a
 * sched_build done at start-up, when allocation was still allowed.
 *
 * The first call on each device also looks up the workspace's device address; make that first call
 * before any stream capture.  All calls on a device share the one workspace (every call
 * overwrites the slices it uses before it reads them): two calls whose kernels may run at the same time on one GPU - different
 * streams, or different host threads - race on it and give wrong results.  Serialise them.
 * Errors: AG_ERR_ARG, AG_ERR_UNSUPPORTED_ARCH, AG_ERR_CUDA; device-side status via ag_last_status.
 */
ag_status gemm_persistent_noalloc(const void* A, const void* B, void* C, int M, int N, int K,
                                  const ag_plan* plan, void* cuda_stream);

/* ---- grouped-query attention decode with die-local KV pages ---------------------------------------
 * Attention is the paper's second scheduled workload (Section 7.1.2; workload appendix: decode = one query token per
 * request, GQA with 8 KV heads, head dimension 128, KV working set 4 B S_k H_kv D bytes).  Work unit = (request, KV
 * head): o = softmax(q K^T / sqrt(D)) V for the H_q / H_kv query heads that share the KV head.  The plan is an ordinary
 * decode-shaped plan with one unit per (request, KV head): sched_build with tile_m = 16, tile_n = 128, k_splits = 1,
 * M = H_q / H_kv, N = 128 * B * H_kv (K is not looked at); unit u = request u / H_kv, KV head u % H_kv.
 * Requests of more than 1024 keys are cut into C = ceil(L / 1024) chunks of 1024 keys, each a unit of its own with its
 * pages on the die that runs it: N = 128 * B * H_kv * C, unit u = ((request * H_kv) + KV head) * C + chunk.  A chunk unit
 * leaves its unnormalised outputs, score maximum and probability sum in a workspace owned by the ag_kv_cache, and a second
 * kernel launched behind the first one puts the chunks of every (request, KV head) together (so two calls on the same
 * ag_kv_cache must not overlap on the GPU).
 */
typedef struct ag_kv_cache ag_kv_cache;
/*
 * ag_kv_pack - store a KV cache in 4 KB pages in the order the tensor cores read them, every unit's pages in chunks
 * of one die (indirect allocation by remapping, Section 7.1.1, applied to the KV cache).
 *   K, V   device, [B][H_kv][L][D] bf16 row-major; D = 128; L a multiple of 128, L <= 2^20
 *   plan   B * H_kv * ceil(L / 1024) units (see above)
 *   amap   affinity map of exactly (dst, dst_bytes), else AG_ERR_STALE_AMAP
 *   dst    device, 4096-aligned; local / remote placement needs room for 2 x the larger die's share, interleaved 1 x
 *   placement  0: on the die that the plan runs the unit on; 1: on the other die; 2: interleaved (consecutive chunks,
 *          the hardware's default placement)
 * Placements 0 and 1 need a map that follows an XOR hash with a free bit (groups of four same-die chunks, see
 * ag_pack_weights_ex), else AG_ERR_NOISY_PROBE.  Synchronises the device.
 * Errors: AG_ERR_ARG, AG_ERR_STALE_AMAP, AG_ERR_NOISY_PROBE, AG_ERR_CUDA, AG_ERR_NOMEM.
 */
ag_status ag_kv_pack(const void* K, const void* V, int B, int H_kv, int L, int D, const ag_plan* plan,
                     const ag_affinity_map* amap, void* dst, size_t dst_bytes, int placement, ag_kv_cache** out);
/* group_free_bit: the hash bit the page groups use (-1: interleaved placement); local_fraction: share of the pages that
 * the map places on the die of their unit (either may be NULL). */
ag_status ag_kv_info(const ag_kv_cache* kv, int32_t* group_free_bit, double* local_fraction);
/*
 * ag_kv_append - write one new token per request into the packed cache (what a decode step does before it attends):
 * the key row and the value row of request b, KV head h go to position pos[b] of that request's pages, i.e. onto the
 * die that the plan of ag_kv_pack runs the unit on.
 *   k_new, v_new  device, [B][H_kv][128] bf16
 *   pos           device [B] int32: 0 <= pos[b] < L, other values leave the request untouched
 * Asynchronous on cuda_stream.  Errors: AG_ERR_ARG, AG_ERR_UNSUPPORTED_ARCH, AG_ERR_CUDA.
 */
ag_status ag_kv_append(ag_kv_cache* kv, const void* k_new, const void* v_new, const int32_t* pos, void* cuda_stream);
void ag_kv_destroy(ag_kv_cache* kv);
/*
 * attention_decode_persistent - O[b][hq][:] = softmax_j(Q[b][hq] . K[b][h][j] / sqrt(D)) V[b][h][j][:], h = hq / (H_q / H_kv),
 * over the first kv_len[b] keys.  Scores and outputs are accumulated in fp32 by tcgen05 MMAs; the probabilities enter
 * the second product as the sum of two bf16 parts (16 significant bits).
 *   Q       device, [B][H_q][128] bf16, 16-byte aligned; H_q / H_kv <= 8
 *   kv      from ag_kv_pack (same B)
 *   kv_len  device [B] int32 or NULL (every request has L keys); values are clamped to 0..L; a request with 0 keys
 *           gets zeros
 *   O       device, [B][H_q][128] fp32, overwritten
 * Asynchronous on cuda_stream.  Errors as gemm_persistent; device-side status via ag_last_status.
 */
ag_status attention_decode_persistent(const void* Q, const ag_kv_cache* kv, const int32_t* kv_len, void* O, int B,
                                      int H_q, const ag_plan* plan, void* cuda_stream);

/*
 * ag_wait_probe - self test of the bounded device-side wait that every kernel of this library
 * uses: one thread waits on a barrier that nothing signals, gives up after limit_ns
 * (<= 1 second) and the call returns AG_ERR_TIMEOUT, with the time actually waited in *waited_ns
 * (host, may be NULL).  The device stays usable.  Errors: AG_ERR_ARG, AG_ERR_UNSUPPORTED_ARCH, AG_ERR_CUDA.
 */
ag_status ag_wait_probe(uint64_t limit_ns, uint64_t* waited_ns);

const char* ag_strerror(ag_status s);
/* A k_splits value for a decode-shaped plan over N weight columns and K rows on sm_budget SMs, from the measurements
 * behind this library (few, large units stream best; without overlapping launches the longest per-SM list sets the time):
 * 4 for N = K = 8192 on 148 SMs with overlapping launches, 8 on 74 SMs, 4 on 37.  overlapping_full_chip: nonzero when the
 * plan uses every SM and policy.overlap_launches is set.  Host arithmetic only; always returns a valid value (>= 1). */
int32_t ag_suggest_k_splits(int32_t N, int32_t K, int32_t sm_budget, int32_t overlapping_full_chip);
/* Last CUDA error code seen by the calling thread inside the library (0 = none). */
int ag_last_cuda_error(void);
/* Number of kernels this library has launched in this process (for launch accounting). */
uint64_t ag_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* ASYMGEMM_H_ */
