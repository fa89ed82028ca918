"""Writes tests/golden/worked_values.txt from exact rational arithmetic.

Uses only ``tests/exact_rational.py`` (integers and fractions): neither the
oracle nor the CUDA library is imported, so the stored values are independent
of both.  Run from the repository root:  python tests/golden/make_worked_values.py
"""
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
sys.path.insert(0, str(HERE.parent))
import exact_rational as R  # noqa: E402

HYP = dict(lr="1e-4", beta1="0.9", beta2="0.999", eps="1e-8", wd="0.1")


def main():
    lines = ["# Worked values of Algorithm 2 and the MCF primitives in exact rational arithmetic",
             "# (tests/golden/make_worked_values.py).  Hex = bfloat16 bit patterns.",
             "# Readings used: eps outside the root, decay product on the first component, one",
             "# rounding per written operator."]
    for t in (1, 2, 3, 10, 100, 1000):
        sc = R.scalars(t=t, **HYP)
        lines.append("scalars t=%d | %s" % (t, " ".join(f"{k}={v:04X}" for k, v in sc.items())))
    for b2 in ("0.999", "0.99", "0.98", "0.95"):
        sc = R.scalars(t=1, **{**HYP, "beta2": b2})
        lines.append(f"beta2 {b2} | {sc['b2h']:04X} {sc['b2l']:04X}")
    prim = [
        ("fast_two_sum 3F80 3A83", R.fast_two_sum(0x3F80, 0x3A83)),
        ("fast_two_sum 4348 3DCD", R.fast_two_sum(0x4348, 0x3DCD)),
        ("two_prod 3F66 3DCD", R.two_prod(0x3F66, 0x3DCD)),
        ("two_prod 3CA4 3CA4", R.two_prod(0x3CA4, 0x3CA4)),
        ("mul 3F80 BA83 3586 0000", R.mcf_mul(0x3F80, 0xBA83, 0x3586, 0x0000)),
        ("scaling 3F66 3F80 BA83", R.scaling(0x3F66, 0x3F80, 0xBA83)),
    ]
    for name, (hi, lo) in prim:
        lines.append(f"{name} | {hi:04X} {lo:04X}")
    # one parameter, theta0 = 0x3CA4, constant gradient 0x3A83, five steps, three strategies
    for strategy in (0, 1, 2):
        th, dth, m, v, dv = 0x3CA4, 0, 0, 0, 0
        for t in range(1, 6):
            sc = R.scalars(t=t, **HYP)
            th, dth, m, v, dv, d = R.adamw_element(th, dth, m, v, dv, 0x3A83, sc, strategy)
            lines.append(f"trace strategy={strategy} t={t} | th={th:04X} dth={dth:04X} m={m:04X} "
                         f"v={v:04X} dv={dv:04X} delta={d:04X}")
    # a second trace with a sign change and epsilon inside the root
    for strategy in (1, 2):
        th, dth, m, v, dv = 0xBF13, 0, 0, 0, 0
        gs = [0x3B21, 0xBA05, 0x3C7F, 0x0000, 0xB9C4, 0x3B21]
        for t, g in enumerate(gs, start=1):
            sc = R.scalars(t=t, **{**HYP, "beta2": "0.95", "lr": "3e-3"})
            th, dth, m, v, dv, d = R.adamw_element(th, dth, m, v, dv, g, sc, strategy, eps_inside=True)
            lines.append(f"trace2 strategy={strategy} t={t} g={g:04X} | th={th:04X} dth={dth:04X} m={m:04X} "
                         f"v={v:04X} dv={dv:04X} delta={d:04X}")
    # "Not updated" (Figure 3, left; Def. 3.2) for a parameter held as an expansion: the effective update of
    # Eq. 2 is zero, decided here on exact rationals.  `lost` is that decision; `components` says whether both
    # stored bit patterns kept their value, a different reading that the cases marked "resplit" tell apart:
    # Grow returns the same value split over other components.  Found by scanning normalised pairs in order.
    picked = {"resplit": [], "kept": [], "moved": []}
    for a in (0x35AB, 0xB5AB, 0x3480, 0xB6C0):
        room = {"resplit": len(picked["resplit"]) + 5, "kept": len(picked["kept"]) + 2, "moved": len(picked["moved"]) + 2}
        for hi in list(range(0x3EF8, 0x3F08)) + list(range(0xBF7C, 0xBF84)):
            for lo in list(range(0x3A00, 0x3B81)) + list(range(0xBA00, 0xBB81)) + [0]:
                if not R.is_normalised(hi, lo):
                    continue
                u, v = R.grow(hi, lo, a)
                same_value = R.value_unchanged(hi, lo, u, v)
                same_bits = R.components_unchanged(hi, lo, u, v)
                kind = "resplit" if same_value and not same_bits else "kept" if same_value else "moved"
                if len(picked[kind]) < room[kind] and (kind != "resplit" or R.is_normalised(u, v)):
                    picked[kind].append((hi, lo, a, u, v, same_value, same_bits))
    for kind in ("resplit", "kept", "moved"):
        for k, (hi, lo, a, u, v, same_value, same_bits) in enumerate(picked[kind]):
            lines.append(f"lost {kind} {k} | x={hi:04X} y={lo:04X} a={a:04X} u={u:04X} v={v:04X} "
                         f"lost={int(same_value)} components={int(same_bits)}")
    (HERE / "worked_values.txt").write_text("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
