/*
 * xstage.h -- host-side calculator for the paper's X-Stage (Burst-Gap) model, C ABI.
 *
 * The model M_X = (T_iss^0, R, Q) (Sec. 3.3): recovered issue floor, effective aggregate drain rate and
 * effective outstanding capacity of a store path, calibrated by microbenchmarks, then applied to a kernel's
 * burst sequence {V_n, T_iss,n^0, G_n}.  All functions are pure host arithmetic in double precision; they
 * allocate nothing and touch no GPU (the one exception, the store microbenchmark at the end, says so).  Units are the caller's, used consistently: bytes, seconds, bytes/second
 * in the examples (the paper's GB is 1e9 bytes, its MiB 2^20 bytes).  [z]_+ means max(z, 0).
 * Pointers are HOST pointers owned by the caller.  Functions returning int return 0 on success and -1 on a bad
 * argument (null pointer, non-positive rate or period, negative count); value-returning functions return NaN
 * on a bad argument.
 */
#ifndef XSTAGE_B200_H_
#define XSTAGE_B200_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  double t_iss0;   /* recovered issue floor T_iss^0 */
  double rate;     /* drain rate R */
  double capacity; /* outstanding capacity Q */
} xstage_params;

/* Eq. 1, the Burst-Gap relation for a periodic pattern of volume V and gap G:
 *   T_period = max(T_iss^0 + G, V/R),   T_iss = max(T_iss^0, V/R - G). */
int xstage_burst_gap(const xstage_params* m, double volume, double gap, double* t_period, double* t_iss);

/* Eq. 2, the smallest gap that returns issue to its floor: G* = [V/R - T_iss^0]_+ . */
double xstage_recovery_gap(const xstage_params* m, double volume);

/* Eq. 6 (first part), occupancy added by one burst issued from a recovered state: b_iso = [V - R T_iss^0]_+ .
 * With the isolated-burst knee volume as V this is the calibration of Q (Sec. 3.5). */
double xstage_isolated_occupancy(const xstage_params* m, double volume);

/*
 * Eqs. 3-6 over a burst sequence (the audit of Sec. 4.1).  For burst n = 0..count-1 with volume[n],
 * floor[n] (its T_iss,n^0; pass NULL to use m->t_iss0 for every burst) and gap[n]:
 *   P_n = floor_n + gap_n,  rho_n = V_n / (R P_n),  delta_b_n = V_n - R P_n,
 *   q_0 = q_initial,  q_{n+1} = [q_n + delta_b_n]_+ ,
 *   guard_n = (q_n + [V_n - R floor_n]_+ <= Q).
 * Outputs (each may be NULL): rho[count], delta_b[count], backlog[count + 1] (q_0..q_count),
 * guard_ok[count] (1 or 0).  Returns the index of the first burst whose guard fails, count if none does,
 * or -1 on a bad argument (P_n must be positive).
 */
int64_t xstage_audit(const xstage_params* m, int64_t count, const double* volume, const double* floor,
                     const double* gap, double q_initial, double* rho, double* delta_b, double* backlog,
                     int32_t* guard_ok);

/* Eq. 7, average gap of the interleaved MegaMoE schedule: G_int = T_L2^mma + (n1/n2) T_L1^mma
 * (the Expert-Wave gap is T_L2^mma alone). */
double xstage_interleaved_gap(double t_l2_mma, double t_l1_mma, double n1, double n2);

/* Eq. 8, issue overhead left after interleaving: [dT_wave - (n1/n2) T_L1^mma]_+ . */
double xstage_interleaved_issue_overhead(double overhead_wave, double t_l1_mma, double n1, double n2);

/* Eq. 9, necessary average-rate condition for full recovery:
 *   n2 V / (n2 (T_iss^0 + T_L2^mma) + n1 T_L1^mma) <= R.   Returns 1, 0, or -1 on a bad argument. */
int xstage_average_rate_feasible(const xstage_params* m, double volume, double t_l2_mma, double t_l1_mma,
                                 double n1, double n2);

/* App. A.2, anti-starvation lead knee: D_knee = ceil(b_n K_SM / (2 h_inter)).  -1 on a bad argument. */
int64_t xstage_lead_knee(int64_t b_n, int64_t k_sm, int64_t h_inter);

/* App. A.2, predicted MMA-side stall: [T_RS - T_cover^mma]_+ . */
double xstage_mma_stall(double t_remote_store_span, double t_cover_mma);

/* App. C.2, tile-aligned sequence length above which the Q-loop gap (at least sigma per K/V tile) covers the
 * recovery gap: M_ub = b_n ceil(G* / sigma).  -1 on a bad argument. */
int64_t xstage_fa_recovery_length(int64_t b_n, double recovery_gap, double sigma);

/*
 * Calibration of M_X from microbenchmark rows (Sec. 3.3 "independent calibration", Sec. 3.5: the three parameters
 * come from the large-gap plateau, the zero-gap runs and the isolated-burst knee).
 *   Periodic rows (one burst volume at several gaps, gap 0 among them): volume, gap, measured issue span t_iss and
 *   period t_period.  Isolated rows (one burst from a recovered state), ascending volume: volume, t_iss.
 *   t_iss0  = median t_iss over the rows whose gap is among the largest third of the distinct gaps (the plateau);
 *   rate    = median of volume / t_period over the rows with gap 0 (drain-limited steady state); 0 if there is none;
 *   the recovered issue floor of an isolated burst grows with its volume (the issue loop itself takes time), so it
 *   is a least-squares line a + b V through the smallest third of the isolated volumes (at least three rows);
 *   the knee is the last row before the first later row whose t_iss exceeds (1 + knee_tolerance)(a + b V);
 *   capacity = [V_knee - rate t_iss(V_knee)]_+   (Eq. 6 from a recovered state).
 * has_knee is 0 (capacity and knee_volume 0) when no row leaves the floor line, when there are fewer than three
 * isolated rows or when there is no zero-gap row.  Returns 0, or -1 on a bad argument (null pointer, no periodic row,
 * negative tolerance, a non-positive period in a zero-gap row).
 */
typedef struct {
  double t_iss0, rate, capacity, knee_volume, floor_intercept, floor_per_byte;
  int32_t has_knee;
} xstage_calibration;

int xstage_calibrate(int64_t n_periodic, const double* p_volume, const double* p_gap, const double* p_t_iss,
                     const double* p_t_period, int64_t n_isolated, const double* i_volume, const double* i_t_iss,
                     double knee_tolerance, xstage_calibration* out);

/*
 * Store microbenchmark on this GPU's own memory: the periodic-burst and isolated-burst patterns of Sec. 3.1, run
 * the way the paper runs its local-memory control (Sec. 3.2), i.e. the identical store kernel with only the
 * destination changed from a peer's memory to this GPU's.  `producers` CTAs of 128 threads, one per SM (producers <= SM count), start together; each
 * repeats `periods` times: issue bytes_per_burst bytes (a multiple of 16) as 16-byte stores into its own slice of
 * device_buffer (DEVICE pointer, 16-byte aligned, buffer_bytes / producers >= bytes_per_burst; slices are walked
 * and wrap, so a buffer well above the L2 size keeps the stores going to HBM), then spin gap_clocks SM clocks
 * without storing.  periods = 1 with gap 0 is an isolated burst from a recovered state.
 * Results, HOST arrays of `periods` doubles, in SM clocks: issue_mean_clocks / issue_max_clocks (may be NULL) =
 * mean / maximum over producers of the sender-visible issue span of burst n (first store issued to last store
 * issued, not completion); period_mean_clocks = mean period n (issue + gap).  *clocks_per_us (may be NULL) = SM
 * clocks per microsecond during the run (clock64 against globaltimer).  Allocates and frees a small device result
 * buffer, runs on the current device, synchronises `stream`.  gap_clocks x periods is limited to 4e9 clocks (about
 * two seconds of spinning on every SM); more is a bad argument.  Returns 0, -1 bad argument, -2 CUDA error,
 * -3 the producers could not be started together within the wait budget.
 */
int xstage_store_probe(int32_t producers, int64_t bytes_per_burst, int64_t gap_clocks, int32_t periods,
                       void* device_buffer, uint64_t buffer_bytes, double* issue_mean_clocks,
                       double* issue_max_clocks, double* period_mean_clocks, double* clocks_per_us, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* XSTAGE_B200_H_ */
