"""Wave-quantized analytical selector: reference implementation (CPU oracle, test infrastructure).

This file is test infrastructure: only the tests, the smoke check and the benchmark's
CPU-baseline leg may import it.  It shares no code with the library's host solver.

It follows the paper's Section III step by step, in the paper's order and notation:
  Eq. 1   R(C) = ceil(C / o_comm)
  Eq. 3   P(C) = o_comp * (G - R(C)); for a kernel family whose compute slot spans `slot_sms` SMs
          (a tile run by a pair of CTAs) only whole slots count: o_comp * floor((G - R(C)) / slot_sms)
  Eq. 5   W_comp = g * (sum_e ceil(M_e / T_M)) * ceil(ceil(N/L) / T_N)
  Eq. 6   V_comp(C) = ceil(W_comp / P(C))
  Eq. 7   W_comm = ceil(ceil(M/D) / T_M^comm) * ceil(ceil(N/L) / T_N^comm)   (per split and rank)
  Eq. 8   V_comm(C) = ceil(W_comm / C)
  Eq. 9   A_s(C) = ceil((s+1) * W_comp / P(C))
  Eq. 10  q(C) = rho * V_comm(C)
  Eq. 11  F_s = max(A_s, F_{s-1}) + q,  F_{-1} = 0
  Eq. 12  T(C) = F_{L-1}
  Eq. 13-15  rho = rho_ref * (K_ref/K) * (T_M,ref*T_N,ref / (T_M*T_N)) * (D/D_ref)
  Algorithm 1  loop over C = 1..C_max, arg min T(C)
  tie breaker  Delta_comp(C) = V_comp(C) * P(C) - W_comp, smaller wins

Readings where the paper is silent (each is listed in the design notes):
  * ties left after Delta_comp go to the smaller C: the winner is the lexicographic
    minimum of (T, Delta_comp, C);
  * candidates with P(C) <= 0 are not in the legal set (Section II-C: the legal set keeps
    positive compute capacity);
  * "the same wave-quantized T(C)" needs exact equality, so rho is quantised once to
    fixed point, rho_q = floor(rho * 2^20 + 1/2), and A_s, q, F_s are carried as integers
    scaled by 2^20;
  * one GPU that emulates all D destination ranks serves every rank's tokens with the same
    C communication CTAs, so the communication work it sees per split is the sum over the
    ranks of Eq. 7 (w_comm_gpu below); Eq. 7 itself is w_comm_rank.

All arithmetic is python int / Fraction: no rounding anywhere except the stated
quantisation of rho.
"""

from __future__ import annotations

from fractions import Fraction

RHO_SHIFT = 20
RHO_ONE = 1 << RHO_SHIFT


def ceil_div(a: int, b: int) -> int:
    return -(-a // b)


# ----------------------------------------------------------------------------- work terms

def w_comp(tiles, g: int, N: int, L: int, T_N: int) -> int:
    """Eq. 5.  `tiles[e]` = ceil(M_e / T_M) (the routed-tile counts, Eq. 16 reduces them)."""
    return g * sum(int(t) for t in tiles) * ceil_div(ceil_div(N, L), T_N)


def normalised_load_tiles(T: int, k_tot: int, E_tot: int, T_M: int) -> list:
    """Section III-E, routed counts left on the device: the selector runs on a normalised-load estimate
    instead of the counts.  The paper gives no formula; the reading taken: the R = T * k_tot
    assignments are spread evenly, every expert holds ceil(R / E_tot) rows, so Eq. 16 sees
    ceil(ceil(R / E_tot) / T_M) tiles per expert."""
    per_expert = ceil_div(T * k_tot, E_tot)
    return [ceil_div(per_expert, T_M)] * E_tot


def w_comm_rank(M: int, D: int, N: int, L: int, T_Mc: int, T_Nc: int) -> int:
    """Eq. 7: communication tiles per split and rank (a rank owns about ceil(M/D) tokens)."""
    return ceil_div(ceil_div(M, D), T_Mc) * ceil_div(ceil_div(N, L), T_Nc)


def owned_tokens(M: int, D: int, d: int) -> int:
    """Tokens owned by rank d when ranks own contiguous blocks of ceil(M/D) tokens."""
    blk = ceil_div(M, D)
    return max(0, min(blk, M - d * blk))


def w_comm_gpu(M: int, D: int, N: int, L: int, T_Mc: int, T_Nc: int) -> int:
    """Communication tiles per split seen by one GPU that emulates all D ranks: the sum
    over the ranks of Eq. 7 evaluated on the tokens each rank really owns."""
    n_col = ceil_div(ceil_div(N, L), T_Nc)
    return sum(ceil_div(owned_tokens(M, D, d), T_Mc) for d in range(D)) * n_col


# ----------------------------------------------------------------------------- rho

def rho_reference(t_comm_us: float, n_splits: int, t_comp_us: float, n_waves: int) -> float:
    """Eq. 13: (time of one communication wave) / (time of one compute wave)."""
    return (t_comm_us / n_splits) / (t_comp_us / n_waves)


def rho_scaled(rho_ref: float, K_ref: int, T_M_ref: int, T_N_ref: int, D_ref: int,
               K: int, T_M: int, T_N: int, D: int) -> float:
    """Eq. 14, evaluated as one product over one product (all factors but rho_ref are
    small integers, so the two products are exact in double precision)."""
    num = float(K_ref * T_M_ref * T_N_ref * D)
    den = float(K * T_M * T_N * D_ref)
    return rho_ref * num / den


def rho_local(rho_ref: float, K_ref: int, T_M_ref: int, T_N_ref: int, rows_ref: int,
              comm_cols_ref: int, K: int, T_M: int, T_N: int, k_tot: int, TP: int,
              N: int, L: int, T_Nc: int) -> float:
    """Re-derivation of Eq. 14 for ranks emulated inside one GPU (Section III-E asks every new
    kernel family for its own service rate): the K and tile-area terms of Eq. 14 stay, the
    ring term D/D_ref goes (nothing crosses a link), and a communication tile costs in
    proportion to the rows moved per token (k_tot*TP read + 1 written) and to its real width
    min(T_N^comm, ceil(N/L))."""
    rows = k_tot * TP + 1
    cols = min(T_Nc, ceil_div(N, L))
    num = float(K_ref * T_M_ref * T_N_ref * rows * cols)
    den = float(K * T_M * T_N * rows_ref * comm_cols_ref)
    return rho_ref * num / den


def quantise_rho(rho: float) -> int:
    """rho_q = floor(rho * 2^20 + 1/2) (rho * 2^20 is exact: a power-of-two scaling)."""
    x = rho * float(RHO_ONE) + 0.5
    return int(x // 1)


# ----------------------------------------------------------------------------- the model

def reservation(C: int, o_comm: int) -> int:
    return ceil_div(C, o_comm)                       # Eq. 1


def compute_capacity(C: int, G: int, o_comp: int, o_comm: int, slot_sms: int = 1) -> int:
    free = G - reservation(C, o_comm)
    return o_comp * (free // slot_sms) if free > 0 else 0     # Eq. 3


def makespan(C: int, Wc: int, Wm: int, L: int, G: int, o_comp: int, o_comm: int, rho, slot_sms: int = 1):
    """T(C) of Eq. 12 with rho any exact number type (int, Fraction).  Returns
    (T, Delta_comp, R, P, [A_s], V_comm) or None when P(C) <= 0."""
    R = reservation(C, o_comm)
    P = compute_capacity(C, G, o_comp, o_comm, slot_sms)
    if P <= 0:
        return None
    A = [ceil_div((s + 1) * Wc, P) for s in range(L)]    # Eq. 9
    V_comm = ceil_div(Wm, C)                              # Eq. 8
    q = rho * V_comm                                      # Eq. 10
    F = 0
    for s in range(L):                                    # Eq. 11
        F = max(A[s], F) + q
    V_comp = ceil_div(Wc, P)                              # Eq. 6
    delta = V_comp * P - Wc                               # tie breaker
    return F, delta, R, P, A, V_comm


def select(Wc: int, Wm: int, L: int, G: int, o_comp: int, o_comm: int, C_max: int, rho_q: int,
           force_comm_ctas: int = 0, selector_off: bool = False, default_C: int = 3,
           slot_sms: int = 1, drain_help: bool = False) -> dict:
    """Algorithm 1 in fixed point.  T_q is T(C) * 2^20 with rho replaced by rho_q / 2^20.

    Precedence (Section III-E): an explicit user value of C wins over everything; with the
    selector switched off the fixed default is used.  Either must be a legal C."""
    def evaluate(C):
        if drain_help:
            m = makespan_drain_help(C, Wc, Wm, L, G, o_comp, o_comm, rho_q, slot_sms)
            if m is None:
                return None
            return dict(comm_ctas=C, R=m[2], P=m[3], T_q=m[0], delta=m[1], W_comp=Wc, W_comm=Wm)
        R = reservation(C, o_comm)
        P = compute_capacity(C, G, o_comp, o_comm, slot_sms)
        if P <= 0:
            return None
        V_comm = ceil_div(Wm, C)
        q = rho_q * V_comm
        F = 0
        for s in range(L):
            A_s = ceil_div((s + 1) * Wc, P)
            F = max(A_s * RHO_ONE, F) + q
        V_comp = ceil_div(Wc, P)
        return dict(comm_ctas=C, R=R, P=P, T_q=F, delta=V_comp * P - Wc,
                    W_comp=Wc, W_comm=Wm)

    if force_comm_ctas > 0 or selector_off:
        C = force_comm_ctas if force_comm_ctas > 0 else default_C
        if C < 1:
            raise ValueError("C must be at least 1")
        r = evaluate(C)
        if r is None:
            raise ValueError("requested C leaves no compute capacity")
        return r
    best = None
    for C in range(1, C_max + 1):
        r = evaluate(C)
        if r is None:
            continue
        key = (r["T_q"], r["delta"], r["comm_ctas"])
        if best is None or key < (best["T_q"], best["delta"], best["comm_ctas"]):
            best = r
    if best is None:
        raise ValueError("no legal C")
    return best


def makespan_drain_help(C: int, Wc: int, Wm: int, L: int, G: int, o_comp: int, o_comm: int, rho_q: int,
                        slot_sms: int = 1):
    """Extension of the recurrence (not in the paper) for a kernel family whose compute CTAs serve
    communication tiles once their GEMM tiles are done.  Fixed point, rho_q = rho * 2^20.
      * splits 0..L-2: Eq. 11 unchanged, C workers;
      * at A_{L-1} (last compute wave over) the tiles still queued -- whole waves of C, at most
        (L-1) W_comm -- plus the last split's W_comm tiles are served by C + H workers, where
        H = P * slot_sms / o_comp is the number of CTAs that were computing.
    Returns (T_q, Delta_comp, R, P) or None when P(C) <= 0."""
    R = reservation(C, o_comm)
    P = compute_capacity(C, G, o_comp, o_comm, slot_sms)
    if P <= 0:
        return None
    q = rho_q * ceil_div(Wm, C)
    F = 0
    for s in range(L - 1):
        F = max(ceil_div((s + 1) * Wc, P) * RHO_ONE, F) + q
    A_last = ceil_div(L * Wc, P) * RHO_ONE
    backlog = 0
    if F > A_last and rho_q > 0:
        backlog = min(ceil_div(F - A_last, rho_q) * C, (L - 1) * Wm)
    workers = C + P * slot_sms // o_comp
    T_q = A_last + rho_q * ceil_div(backlog + Wm, workers)
    return T_q, ceil_div(Wc, P) * P - Wc, R, P


def curve(Wc: int, Wm: int, L: int, G: int, o_comp: int, o_comm: int, C_max: int, rho, slot_sms: int = 1) -> dict:
    """{C: (T, Delta_comp)} for every legal C, rho exact (Fraction or int)."""
    out = {}
    for C in range(1, C_max + 1):
        m = makespan(C, Wc, Wm, L, G, o_comp, o_comm, rho, slot_sms)
        if m is not None:
            out[C] = (m[0], m[1])
    return out


# ----------------------------------------------------------------------------- simulator

def simulate(C: int, Wc: int, Wm: int, L: int, P: int, rho: Fraction) -> dict:
    """Tiny discrete-event simulation of the pipeline the model describes (Section III-C):
      * P compute CTAs; CTA b takes global tiles b, b+P, b+2P, ... of the split-major
        sequence (L splits of Wc tiles each); every tile takes one time unit;
      * split s is published when its last tile has finished;
      * C communication CTAs serve the splits in order; for one split, CTA c takes
        communication tiles c, c+C, ...; every communication tile takes rho time units and
        the CTAs move to the next split together (a split is served in waves);
      * service of split s starts when it is published and split s-1 has been served.
    Returns the publication times and the finish times, computed event by event (no
    closed form is used)."""
    rho = Fraction(rho)
    # compute side: per-CTA clocks
    clock = [Fraction(0)] * P
    tile_end = [None] * (L * Wc)
    for i in range(L * Wc):
        b = i % P
        clock[b] = clock[b] + 1
        tile_end[i] = clock[b]
    publish = []
    for s in range(L):
        seg = tile_end[s * Wc:(s + 1) * Wc]
        publish.append(max(seg) if seg else Fraction(0))
    # communication side
    finish = []
    prev = Fraction(0)
    for s in range(L):
        start = max(publish[s], prev)
        worker = [start] * C
        for j in range(Wm):
            c = j % C
            worker[c] = worker[c] + rho
        prev = max(worker) if Wm > 0 else start
        finish.append(prev)
    return dict(publish=publish, finish=finish, T=finish[-1] if finish else Fraction(0))


def simulate_drain_help(C: int, Wc: int, Wm: int, L: int, P: int, helpers: int, rho: Fraction) -> dict:
    """Event-by-event simulation of the schedule the drain-help model stands for (no closed form):
      * compute side as in simulate();
      * the C communication CTAs serve splits 0..L-2 in order, each split in waves of at most C tiles,
        a wave takes rho;
      * at A = the publication time of the last split every wave of those splits that has not
        completed goes back to the pool with the tiles it really holds, together with the last
        split's Wm tiles; the pool is served by C + helpers workers, rho per tile, from time A.
    The model (makespan_drain_help) counts C tiles for every wave that is still open at A and counts
    idle gaps between splits as waves, so it can only over-estimate this simulation; the two agree
    when nothing is open at A, and when the service up to A is gap-free and Wm is a multiple of C."""
    rho = Fraction(rho)
    clock = [Fraction(0)] * P
    tile_end = []
    for i in range(L * Wc):
        b = i % P
        clock[b] = clock[b] + 1
        tile_end.append(clock[b])
    publish = []
    for s in range(L):
        seg = tile_end[s * Wc:(s + 1) * Wc]
        publish.append(max(seg) if seg else Fraction(0))
    A = publish[L - 1]
    pool = Wm
    prev = Fraction(0)
    gap_free = True
    for s in range(L - 1):
        start = max(publish[s], prev)
        if s > 0 and publish[s] > prev:
            gap_free = False
        left, t = Wm, start
        while left > 0:
            n = min(C, left)
            if t + rho > A:          # this wave is not complete at A: its tiles are pooled
                pool += n
            t += rho
            left -= n
        prev = t
    workers = C + helpers
    worker = [A] * workers
    for j in range(pool):
        worker[j % workers] += rho
    T = max(worker) if pool > 0 else A
    return dict(publish=publish, T=T, pool=pool, gap_free=gap_free, open_at_A=pool > Wm)



# ----------------------------------------------------------------------------- co-resident family
# Re-derivation for a kernel family in which communication work shares SMs with compute (Section III-B
# lets o_comm exceed 1; Section III-E asks a new kernel family to re-derive o_comp, o_comm, tile work, the
# dependency recurrence, the legal range and the service rate).  Not in the paper: this library's own
# extension, pinned by its reductions to the recurrences above, closed forms, hand-worked values and an
# event simulation (tests/test_oracle_solver.py).
#
#   * the unit of communication capacity is a WARP.  A dedicated communication CTA is `warps_cta` warps;
#     a compute CTA carries w co-resident communication warps (the second decision variable) and turns
#     into `warps_cta` communication warps once its GEMM tiles are done (drain help);
#   * a communication tile is handed out in `quanta_tile` pieces ("quanta": one per warp of a dedicated CTA
#     under the static map, one per token of the tile under the kernels' dynamic hand-out); one warp serves a
#     quantum in rho * warps_cta / quanta_tile, so that a dedicated CTA still serves a tile in rho compute
#     waves (Eq. 10 with quanta and warps in place of tiles and CTAs);
#   * bandwidth-coupled service rate: N warps streaming together are limited by HBM once N exceeds `n_sat`
#     (the warp count whose aggregate demand equals the measured copy bandwidth); the time of one quantum is
#     rho(N) = rho * max(N, n_sat) / n_sat (rounded up in fixed point);
#   * a co-resident warp shares its SM's issue slots and memory path with a running GEMM: it serves
#     `gamma` times slower than a dedicated warp (N_eff counts it as 1/gamma warps), and every co-resident
#     warp stretches the compute wave by `beta`; with more than one split they also force the split-major
#     tile order (x is read once per split), which stretches the compute wave by `order`;
#   * without co-resident warps the kernels run the tiles m-tile-major across the splits (x is read once):
#     no split is published before the last one, so for w = 0 every split becomes ready at A_{L-1} and all
#     communication work is served after the GEMM (dedicated CTAs then only cost SMs).
#   All four constants are fixed point (2^-20) except n_sat and warps_cta (integers).

def coupled_rho(rho_q: int, n_workers: int, n_sat: int) -> int:
    """rho(N) = rho * max(N, n_sat) / n_sat, rounded up to the next multiple of 2^-20."""
    return ceil_div(rho_q * max(n_workers, n_sat), n_sat)


def coupled_service(rho_q: int, quanta: int, n_workers: int, n_sat: int) -> int:
    """Time to serve `quanta` with n_workers warps, in waves of n_workers: a wave in which n warps stream
    together takes rho(n), so the full waves take rho(n_workers) each and a last partial wave of r quanta
    takes rho(r).  Below saturation this is Eq. 8 and Eq. 10, rho * ceil(quanta / n_workers); far above it
    it tends to rho * quanta / n_sat: the bytes at the bandwidth, however many warps share them."""
    full, rest = divmod(quanta, n_workers)
    return full * coupled_rho(rho_q, n_workers, n_sat) + (coupled_rho(rho_q, rest, n_sat) if rest else 0)


def makespan_co_resident(C: int, w: int, Wc: int, Wm: int, L: int, G: int, o_comp: int, o_comm: int, rho_q: int,
                         slot_sms: int, warps_cta: int, n_sat: int, beta_q: int, gamma_q: int, order_q: int,
                         quanta_tile: int = 0):
    """T(C, w) for the co-resident family with drain help, fixed point.  `quanta_tile` = pieces a
    communication tile is handed out in (0: one per warp of a dedicated CTA, `warps_cta`; the dynamic
    hand-out of the kernels gives out single tokens of a tile, T_M^comm pieces): one warp serves one piece in
    rho * warps_cta / quanta_tile (rounded down in fixed point), so that a dedicated CTA still serves a tile
    in rho.  Returns (T_q, Delta_comp, R, P) or None when P(C) <= 0."""
    R = reservation(C, o_comm)
    P = compute_capacity(C, G, o_comp, o_comm, slot_sms)
    if P <= 0:
        return None
    if quanta_tile > 0:
        rho_q = rho_q * warps_cta // quanta_tile               # service time of one piece by one warp
    else:
        quanta_tile = warps_cta
    n_sm = P * slot_sms // o_comp                              # SMs that compute
    tau_q = RHO_ONE + w * beta_q + (order_q if (w > 0 and L > 1) else 0)     # one compute wave
    Wq = Wm * quanta_tile                                      # quanta per split
    n_early = C * warps_cta + w * n_sm                         # warps that serve while the GEMM runs
    n_eff = C * warps_cta + (w * n_sm * RHO_ONE) // gamma_q    # ... in dedicated-warp equivalents
    A_last = ceil_div(L * Wc, P) * tau_q
    if n_eff <= 0:
        backlog = (L - 1) * Wq                                 # nobody serves before the GEMM is over
    else:
        q_wave = coupled_rho(rho_q, n_early, n_sat)
        q = q_wave * ceil_div(Wq, n_eff)
        F = 0
        for s in range(L - 1):                                 # Eq. 11 on splits 0..L-2
            A_s = ceil_div((s + 1) * Wc, P) * tau_q if w > 0 else A_last     # m-tile-major order: nothing is early
            F = max(A_s, F) + q
        backlog = 0
        if F > A_last and q_wave > 0:
            backlog = min(ceil_div(F - A_last, q_wave) * n_eff, (L - 1) * Wq)
    n_tail = (C + n_sm) * warps_cta + w * n_sm                 # every warp serves once the GEMM is over
    T_q = A_last + coupled_service(rho_q, backlog + Wq, n_tail, n_sat)
    return T_q, ceil_div(Wc, P) * P - Wc, R, P


def select_co_resident(Wc: int, Wm: int, L: int, G: int, o_comp: int, o_comm: int, C_max: int, rho_q: int,
                       slot_sms: int, w_max: int, C_co_max: int, warps_cta: int, n_sat: int, beta_q: int,
                       gamma_q: int, order_q: int, force_comm_ctas: int = 0, selector_off: bool = False,
                       default_C: int = 3, force_co_warps: int = -1, quanta_tile: int = 0,
                       co_min_waves: int = 0) -> dict:
    """Algorithm 1 over the product set: C in 1..C_max with w = 0, and C in 1..min(C_max, C_co_max) with
    w in 1..w_max (a one-time characterisation bounds the dedicated CTAs worth trying beside co-resident
    warps, as the paper's C <= 16 does for its family).  A second characterisation constant bounds the
    legal set from below: co-resident warps are only legal when the compute phase is at least
    `co_min_waves` waves long, ceil(L * W_comp / P(C)) >= co_min_waves (on shorter launches their start-up
    costs more than they can overlap, which a wave model does not see).  Lexicographic minimum of
    (T, Delta_comp, w, C).  Overrides as in select(): a forced C / a forced w restrict the set to that value
    (a forced w is not subject to co_min_waves)."""
    if force_comm_ctas > 0 or selector_off:
        Cs0 = Cs1 = [force_comm_ctas if force_comm_ctas > 0 else default_C]
        if Cs0[0] < 1:
            raise ValueError("C must be at least 1")
    else:
        Cs0 = list(range(1, C_max + 1))
        Cs1 = list(range(1, min(C_max, C_co_max) + 1))
    ws = list(range(0, w_max + 1)) if force_co_warps < 0 else [min(force_co_warps, w_max)]
    best = None
    for w in ws:
        for C in (Cs0 if w == 0 else Cs1):
            m = makespan_co_resident(C, w, Wc, Wm, L, G, o_comp, o_comm, rho_q, slot_sms, warps_cta, n_sat,
                                     beta_q, gamma_q, order_q, quanta_tile)
            if m is None:
                continue
            if w > 0 and force_co_warps < 0 and ceil_div(L * Wc, m[3]) < co_min_waves:
                continue
            key = (m[0], m[1], w, C)
            if best is None or key < best[0]:
                best = (key, dict(comm_ctas=C, co_warps=w, R=m[2], P=m[3], T_q=m[0], delta=m[1], W_comp=Wc, W_comm=Wm))
    if best is None:
        raise ValueError("no legal (C, w)")
    return best[1]


def simulate_co_resident(C: int, w: int, Wc: int, Wm: int, L: int, P: int, n_sm: int, rho: Fraction,
                         warps_cta: int, n_sat: int, beta: Fraction, gamma: Fraction, order: Fraction,
                         quanta_tile: int = 0) -> dict:
    """Event-by-event simulation of the schedule makespan_co_resident stands for (no closed form):
      * P compute slots take tiles round-robin, a tile takes tau = 1 + w*beta (+ order when w > 0 and L > 1);
      * while the GEMM runs, split s (once published, and after split s-1) is served in waves of at most
        n_eff = C*warps_cta + floor(w*n_sm/gamma) quanta, a wave takes rho * max(N_early, n_sat) / n_sat;
      * at A = the publication of the last split every wave that has not completed returns its quanta to
        the pool, which with the last split's quanta is served by all N_tail warps, wave by wave; a wave in
        which n warps stream together takes rho * max(n, n_sat) / n_sat.
    As with simulate_drain_help the closed form can only over-estimate (it counts an open wave in full)."""
    rho, beta, gamma, order = Fraction(rho), Fraction(beta), Fraction(gamma), Fraction(order)
    if quanta_tile > 0:
        rho = rho * warps_cta / quanta_tile        # one warp, one quantum
    else:
        quanta_tile = warps_cta
    tau = 1 + w * beta + (order if (w > 0 and L > 1) else 0)
    clock = [Fraction(0)] * P
    tile_end = []
    for i in range(L * Wc):
        b = i % P
        clock[b] += tau
        tile_end.append(clock[b])
    publish = [max(tile_end[s * Wc:(s + 1) * Wc]) if Wc > 0 else Fraction(0) for s in range(L)]
    A = publish[L - 1]
    if w == 0:
        publish = [A] * L                  # m-tile-major order: every split completes with the last tile
    Wq = Wm * quanta_tile
    n_early = C * warps_cta + w * n_sm
    n_eff = C * warps_cta + int(Fraction(w * n_sm) / gamma)
    pool = Wq
    open_at_A = False
    if n_eff <= 0:
        pool += (L - 1) * Wq
    else:
        wave = rho * max(n_early, n_sat) / n_sat
        prev = Fraction(0)
        for s in range(L - 1):
            t = max(publish[s], prev)
            left = Wq
            while left > 0:
                n = min(n_eff, left)
                if t + wave > A:
                    pool += n
                    open_at_A = True
                t += wave
                left -= n
            prev = t
    n_tail = (C + n_sm) * warps_cta + w * n_sm
    T = A
    left = pool
    while left > 0:                       # wave by wave: n warps streaming together take rho * max(n, n_sat) / n_sat
        n = min(n_tail, left)
        T += rho * max(n, n_sat) / n_sat
        left -= n
    return dict(publish=publish, T=T, pool=pool, open_at_A=open_at_A)


# ----------------------------------------------------------------------------- tile-level readiness
# Section III-C derives A_s from the position of a split's LAST tile in the global tile sequence (Eq. 9):
# readiness is one number per split.  A kernel that publishes every tile lets a communication tile start
# as soon as the compute tiles under ITS tokens are done.  The same construction as Eq. 9, applied to each
# communication tile instead of each split:
#   * inside a split the compute tiles run expert by expert, m-tile by m-tile (index (mu*g + p)*NT + n);
#   * the rows of an expert are in token order (stable sort), so the tokens of the communication token-tile
#     that ends at token t_hi sit in the last non-empty expert's rows up to about M_e * t_hi / T (its load
#     taken as even over the tokens: exact for an always-active shared expert), i.e. in its m-tiles up to
#     i = ceil(n_last * t_hi / T) - 1 of its n_last tiles; every earlier expert's tiles come before those;
#   * the communication tile (token-tile j, column tile c) is therefore complete when compute tile
#       idx(j, c) = ((S - n_last + i_j) * g + (g - 1)) * NT + n_hi(c)
#     of its split has finished, at the end of wave floor((s*W_comp + idx) / P), one more than that in
#     compute-wave units (Eq. 9 is the special case idx = W_comp - 1).
# Not in the paper as an equation: this library's reading of "split-level dependency" for per-tile flags.

def comm_tile_ready_index(tiles, g: int, M: int, D: int, N: int, L: int, T_N: int, T_Mc: int, T_Nc: int) -> list:
    """idx(j, c) for every communication tile of a split, in the static map's order ct = j * n_col + c
    (token-tiles rank-major: rank d owns a contiguous block of ceil(M/D) tokens)."""
    tiles = [int(t) for t in tiles]
    S = sum(tiles)
    split_w = ceil_div(N, L)
    NT = ceil_div(split_w, T_N)
    n_col = ceil_div(split_w, T_Nc)
    nz = [t for t in tiles if t > 0]
    n_last = nz[-1] if nz else 0
    blk = ceil_div(M, D)
    out = []
    for d in range(D):
        own = owned_tokens(M, D, d)
        for ti in range(ceil_div(own, T_Mc)):
            t_hi = d * blk + min(own, (ti + 1) * T_Mc)
            i_j = max(0, ceil_div(n_last * t_hi, M) - 1) if M > 0 else 0
            mu = S - n_last + i_j
            for c in range(n_col):
                n_hi = ceil_div(min(split_w, (c + 1) * T_Nc), T_N) - 1
                out.append((mu * g + (g - 1)) * NT + n_hi)
    return out


def makespan_tile_level(C: int, ready_idx, Wc: int, L: int, G: int, o_comp: int, o_comm: int, rho, slot_sms: int = 1):
    """The static partition (Section III-A map: communication tile ct belongs to CTA ct mod C) with
    tile-level readiness, wave by wave: wave v of split s (tiles vC .. vC+C-1) starts when all its tiles
    are ready and the previous wave is served,
        F_{s,v} = max(max_{ct < min(vC+C, W_comm)} a_{s,ct}, F_{s,v-1}) + rho,   T = F_{L-1, V-1},
    a_{s,ct} = floor((s W_comp + idx(ct)) / P) + 1 (the maximum may run over all earlier tiles of the split
    as well: their waves have been served by then).  rho exact (int scaled by 2^20, or Fraction).
    Returns (T, Delta_comp, R, P) or None when P(C) <= 0."""
    R = reservation(C, o_comm)
    P = compute_capacity(C, G, o_comp, o_comm, slot_sms)
    if P <= 0:
        return None
    Wm = len(ready_idx)
    one = RHO_ONE if isinstance(rho, int) else 1
    F = 0
    for s in range(L):
        top = -1                                   # largest idx among the tiles of this split seen so far
        for v in range(ceil_div(Wm, C)):
            top = max([top] + list(ready_idx[v * C:min(v * C + C, Wm)]))
            a = ((s * Wc + top) // P + 1) * one
            F = max(a, F) + rho
    return F, ceil_div(Wc, P) * P - Wc, R, P


def simulate_tile_level(C: int, ready_idx, Wc: int, L: int, P: int, rho: Fraction) -> dict:
    """Event simulation of the static partition with per-tile flags, CTA by CTA (no waves): compute CTA b
    takes global tiles b, b+P, ... (unit time each); communication CTA k walks its tiles k, k+C, ... of
    split 0, then of split 1, ...; a tile starts when the compute tile idx(ct) of its split has finished and
    the CTA is free, and takes rho."""
    rho = Fraction(rho)
    clock = [Fraction(0)] * P
    tile_end = []
    for i in range(L * Wc):
        b = i % P
        clock[b] += 1
        tile_end.append(clock[b])
    Wm = len(ready_idx)
    worker = [Fraction(0)] * C
    for s in range(L):
        for ct in range(Wm):
            k = ct % C
            worker[k] = max(worker[k], tile_end[s * Wc + ready_idx[ct]]) + rho
    return dict(T=max(worker) if Wm > 0 and L > 0 else Fraction(0))
