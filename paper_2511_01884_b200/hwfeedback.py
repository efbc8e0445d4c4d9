"""Hardware feedback the way the paper prepares it for its Judge (Section 2.3, Algorithms 1-2,
Appendix C): read Nsight Compute metrics of profiled kernels, reduce them to the 24-metric key
subset, and -- off line -- select the metrics that track kernel runtime across tasks.

    python -m paper_2511_01884_b200.hwfeedback metrics                     # the list, for ``ncu --metrics``
    python -m paper_2511_01884_b200.hwfeedback key24 report.csv            # the key subset of one capture
    python -m paper_2511_01884_b200.hwfeedback select taskA/*.csv -- taskB/*.csv ...

``report.csv`` is the output of ``ncu -i <file>.ncu-rep --page raw --csv`` (one row per profiled
launch, one column per metric).  Host-side tooling only: nothing here runs on the GPU or is used by
the operator's kernels.

Selection (Section 2.3, steps 2 and 3), for tasks i = 1..n, each with the metric table of its
profiled kernel variants and their runtimes:
  step 2   r[m, i] = Pearson correlation of metric m with runtime over the kernels of task i;
           the candidates of task i are its 20 metrics of largest |r| (aliases and collinear
           duplicates removed first);
  step 3   S[m] = (1/n) sum_i |r[m, i]| over all tasks; keep the metrics that are candidates of
           more than one task, whose correlation has the same sign in every task where it is
           defined, and whose S[m] exceeds the 75th percentile of S over all candidates.
"""
from __future__ import annotations

import csv
import io
import sys
from typing import Dict, Iterable, List, Mapping, Optional, Sequence, Tuple

import numpy as np

# The key subset of Appendix C ("The 24-metric key subset"), in the paper's order.  These are
# Nsight Compute metric identifiers, i.e. an interface: they have to be spelled as the tool
# spells them.
KEY24: Tuple[str, ...] = (
    "sm__cycles_active.avg",
    "sm__warps_active.avg.pct_of_peak_sustained_active",
    "launch__occupancy_limit_blocks",
    "launch__occupancy_limit_registers",
    "launch__occupancy_limit_shared_mem",
    "launch__registers_per_thread",
    "sm__inst_executed.sum",
    "sm__inst_executed_pipe_fp32.avg.pct_of_peak_sustained_active",
    "sm__inst_executed_pipe_tensor.avg.pct_of_peak_sustained_active",
    "dram__bytes_read.sum",
    "dram__bytes_write.sum",
    "dram__throughput.avg.pct_of_peak_sustained_elapsed",
    "dram__bytes.sum.per_second",
    "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed",
    "l1tex__t_sector_hit_rate.pct",
    "l1tex__throughput.avg.pct_of_peak_sustained_active",
    "lts__t_sector_hit_rate.pct",
    "lts__throughput.avg.pct_of_peak_sustained_active",
    "smsp__warp_issue_stalled_memory_dependency_per_warp_active.pct",
    "smsp__warp_issue_stalled_short_scoreboard_per_warp_active.pct",
    "smsp__warp_issue_stalled_long_scoreboard_per_warp_active.pct",
    "smsp__warp_issue_stalled_barrier_per_warp_active.pct",
    "smsp__warp_issue_stalled_branch_resolving_per_warp_active.pct",
    "smsp__sass_average_branch_targets_threads_uniform.pct",
)
RUNTIME_METRIC = "gpu__time_duration.sum"

# decimal prefixes Nsight Compute puts on units when it scales a value for display
_SCALE = {"K": 1e3, "M": 1e6, "G": 1e9, "T": 1e12, "m": 1e-3, "u": 1e-6, "n": 1e-9}
_BASE_UNITS = ("byte", "byte/s", "cycle", "inst", "hz", "s", "second", "sector", "request", "warp", "thread", "block", "register/thread")


def _to_base(value: float, unit: str) -> float:
    """Undo the display scaling of a unit such as ``Gbyte``, ``us``, ``Tbyte/s`` or ``Ghz``."""
    u = unit.strip()
    low = u.lower()
    for base in _BASE_UNITS:
        if low == base:
            return value
        if len(u) == len(base) + 1 and low[1:] == base and u[0] in _SCALE:
            return value * _SCALE[u[0]]
    return value


def read_ncu_raw_csv(text: str) -> List[Dict[str, float]]:
    """One dict {metric name: value in base units} per profiled launch.  Non-numeric columns
    (kernel name, device ...) are kept as strings under their header."""
    rows = list(csv.reader(io.StringIO(text)))
    rows = [r for r in rows if r and not r[0].startswith("==")]
    if len(rows) < 3:
        raise ValueError("expected a header row, a unit row and at least one launch")
    header, units = rows[0], rows[1]
    out = []
    for r in rows[2:]:
        d: Dict[str, float] = {}
        for name, unit, cell in zip(header, units, r):
            try:
                d[name] = _to_base(float(cell.replace(",", "")), unit)
            except ValueError:
                d[name] = cell            # type: ignore[assignment]
        out.append(d)
    return out


def key24(metrics: Mapping[str, float]) -> List[Tuple[int, str, Optional[float]]]:
    """(number in the paper's table, name, value or None when the capture does not hold it)."""
    return [(i + 1, m, metrics[m] if isinstance(metrics.get(m), float) else None) for i, m in enumerate(KEY24)]


# ---- selection ---------------------------------------------------------------------------------
def pearson(x: Sequence[float], y: Sequence[float]) -> float:
    """Pearson correlation coefficient; nan when either sample has no variance."""
    a = np.asarray(x, dtype=np.float64)
    b = np.asarray(y, dtype=np.float64)
    if a.shape != b.shape or a.ndim != 1 or a.size < 2:
        raise ValueError("two equally long samples of at least two values are required")
    da, db = a - a.mean(), b - b.mean()
    den = np.sqrt((da * da).sum() * (db * db).sum())
    if den == 0.0 or not np.isfinite(den):
        return float("nan")
    return float((da * db).sum() / den)


def drop_collinear(table: Mapping[str, Sequence[float]], threshold: float = 0.999) -> List[str]:
    """Names of ``table`` in order, without constant or non-finite columns and without a column whose
    |correlation| with an earlier kept column reaches ``threshold`` (aliases of one counter)."""
    kept: List[str] = []
    cols: List[np.ndarray] = []
    for name, col in table.items():
        c = np.asarray(col, dtype=np.float64)
        if not np.isfinite(c).all() or np.ptp(c) == 0.0:
            continue
        z = (c - c.mean()) / np.sqrt(((c - c.mean()) ** 2).sum())
        if any(abs(float(z @ k)) >= threshold for k in cols):
            continue
        kept.append(name)
        cols.append(z)
    return kept


def task_correlations(table: Mapping[str, Sequence[float]], runtime: Sequence[float], top: int = 20,
                      collinear: float = 0.999) -> Tuple[Dict[str, float], List[str]]:
    """Step 2 for one task: ({metric: r with runtime}, the ``top`` metrics of largest |r|)."""
    # the runtime column itself takes no part: a counter that is collinear with runtime (active
    # cycles, the first entry of the paper's subset) is a candidate, not an alias to drop
    names = drop_collinear({m: c for m, c in table.items() if m != RUNTIME_METRIC}, collinear)
    r = {m: pearson(table[m], runtime) for m in names}
    r = {m: v for m, v in r.items() if np.isfinite(v)}
    ranked = sorted(r, key=lambda m: (-abs(r[m]), m))
    return r, ranked[:top]


def select_across_tasks(per_task: Sequence[Tuple[Mapping[str, float], Sequence[str]]]) -> Dict[str, object]:
    """Step 3.  ``per_task`` holds the (correlations, candidates) pair of every task.  Returns the
    global scores of all candidates, their 75th percentile and the selected metrics (sorted by score)."""
    n = len(per_task)
    if n == 0:
        raise ValueError("no task")
    candidates = sorted({m for _, top in per_task for m in top})
    score, sign_ok, count = {}, {}, {}
    for m in candidates:
        rs = [r[m] for r, _ in per_task if m in r]
        score[m] = sum(abs(v) for v in rs) / n          # a task where r is undefined contributes 0
        sign_ok[m] = all(v > 0 for v in rs) or all(v < 0 for v in rs)
        count[m] = sum(1 for _, top in per_task if m in top)
    p75 = float(np.percentile(list(score.values()), 75)) if score else float("nan")
    chosen = [m for m in candidates if count[m] > 1 and sign_ok[m] and score[m] > p75]
    chosen.sort(key=lambda m: (-score[m], m))
    return {"scores": score, "p75": p75, "selected": chosen, "appearances": count, "same_sign": sign_ok}


def tables_from_reports(launches: Iterable[Mapping[str, float]]) -> Tuple[Dict[str, List[float]], List[float]]:
    """Metric table and runtimes of one task from the parsed launches of its kernel variants
    (only metrics that every launch reports as a number are kept)."""
    launches = list(launches)
    common = [m for m in launches[0] if all(isinstance(l.get(m), float) for l in launches)]
    table = {m: [l[m] for l in launches] for m in common}
    return table, table[RUNTIME_METRIC]


def _main(argv: List[str]) -> int:
    if argv[:1] == ["metrics"]:
        print(",".join(KEY24 + (RUNTIME_METRIC,)))
        return 0
    if len(argv) >= 2 and argv[0] == "key24":
        for path in argv[1:]:
            for launch in read_ncu_raw_csv(open(path).read()):
                print(f"# {launch.get('Kernel Name', '?')}  ({path})")
                for i, name, v in key24(launch):
                    print(f"{i:2d}  {name:70s} {'not reported' if v is None else f'{v:.6g}'}")
        return 0
    if len(argv) >= 2 and argv[0] == "select":
        groups, cur = [], []
        for a in argv[1:]:
            if a == "--":
                groups.append(cur)
                cur = []
            else:
                cur.append(a)
        groups.append(cur)
        per_task = []
        for g in groups:
            launches = [l for path in g for l in read_ncu_raw_csv(open(path).read())]
            table, runtime = tables_from_reports(launches)
            per_task.append(task_correlations(table, runtime))
        res = select_across_tasks(per_task)
        print(f"{len(res['scores'])} candidates over {len(groups)} tasks, P75 of the global score = {res['p75']:.4f}")
        for m in res["selected"]:
            print(f"{res['scores'][m]:.4f}  {m}" + ("   [key-24]" if m in KEY24 else ""))
        return 0
    print(__doc__)
    return 2


if __name__ == "__main__":
    raise SystemExit(_main(sys.argv[1:]))
