"""Markdown table of the five configs from the records a GPU run leaves behind.

  python -m paper_2504_13818_b200.report <all_configs.json> <parity_maxima.jsonl>

<all_configs.json> is the line `python bench.py --all-configs` prints; <parity_maxima.jsonl> is the file the `-m gpu`
tests append to (PODS_PARITY_RECORD; one JSON object per parity case with the maxima they achieved).  Reads the two files and
prints; computes nothing of the method."""
import json
import sys


def _fmt(x, digits=3):
    if x is None:
        return ""
    if isinstance(x, float):
        return ("%." + str(digits) + "g") % x
    return str(x)


def parity_by_config(path):
    """Worst recorded maxima per config name (the case strings start with the workload's name)."""
    out = {}
    try:
        lines = open(path).read().splitlines()
    except OSError:
        return out
    for line in lines:
        try:
            d = json.loads(line)
        except ValueError:
            continue
        case = d.get("case", "")
        for name in ("c1_tiny", "c2_qwen_vocab", "c3_select_mixed", "c4_select_ties", "c5_large_loss"):
            if case.startswith(name):
                cur = out.setdefault(name, {})
                for k, v in d.items():
                    if isinstance(v, (int, float)) and k not in ("V", "rows", "loss", "loss_term_scale"):
                        cur[k] = max(cur.get(k, 0), v)
    return out


def main(argv):
    rec = json.loads(open(argv[1]).read().strip().splitlines()[-1])
    par = parity_by_config(argv[2]) if len(argv) > 2 else {}
    peak = rec["hbm_peak_GBps"]
    print("| Config | select: groups/s (us; GB/s; %% of %.0f; %% of 8000) | oracle groups/s (cores) | loss+grad: tokens/s "
          "(kernel GB/s; %% of %.0f; %% of 8000) | oracle tokens/s (cores) | idx | max adv rel | max logp abs | loss rel "
          "(literal / conditioned) | max dlogits ulp (rows with allowance) |" % (peak, peak))
    print("|---|---|---|---|---|---|---|---|---|---|")
    for e in rec["all_configs"]:
        s, l = e["select"], e.get("loss")
        p = par.get(e["workload"], {})
        sel = "%s (%.1f; %.0f; %.1f; %.1f)" % (_fmt(s["groups_per_s"]), s["us"], s["GBps"], 100 * s["frac_of_measured_hbm"],
                                                100 * s["frac_of_nominal_8TBps"])
        loss = ""
        orc = ""
        if l:
            loss = "%s (%.0f; %.1f; %.1f)" % (_fmt(l["tokens_per_s_step"]), l["GBps_loss_kernel"],
                                              100 * l["frac_of_measured_hbm"], 100 * l["frac_of_nominal_8TBps"])
            orc = "%s (%d)" % (_fmt(l["oracle_tokens_per_s"]), l["oracle_cores"])
        lossrel = ""
        if "loss_rel_literal" in p or "share_rel_literal" in p:
            lossrel = "%s / %s" % (_fmt(p.get("loss_rel_literal", p.get("share_rel_literal")), 2),
                                   _fmt(p.get("loss_rel_conditioned", p.get("share_rel_conditioned")), 2))
        dl = ""
        if "literal_ulps" in p:
            dl = "%s (%d)" % (_fmt(p["literal_ulps"], 2), p.get("allowance_rows", 0))
        print("| %s | %s | %s (%d) | %s | %s | %s | %s | %s | %s | %s |" % (
            e["workload"], sel, _fmt(s["oracle_groups_per_s"]), s["oracle_cores"], loss, orc,
            "exact" if p.get("idx_exact") else "", _fmt(p.get("adv_rel"), 2),
            _fmt(p.get("logp_abs", p.get("logp_abs_all_rows")), 2), lossrel, dl))


if __name__ == "__main__":
    main(sys.argv)
