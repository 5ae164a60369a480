"""The pins must be able to fail: each plausible slip, planted in a copy of the oracle's source, has to
break at least one of them.  (The real oracle is untouched: the altered copy is compiled elsewhere.)"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "cascade_oracle.cpp")
PINS = ["test_oracle_plan_first.py", "test_oracle_budget.py", "test_oracle_schedule.py", "test_oracle_plan.py", "test_oracle_copy.py",
        "test_oracle_prefetch.py", "test_oracle_policies.py", "test_oracle_more_pins.py"]

DEEP_PINS = ["test_oracle_deep.py"]

MUTATIONS = [
    ("eq3 drops the one half", "const int64_t L = ((L_act + L_max) * p->gamma_q16) >> 17;",
     "const int64_t L = ((L_act + L_max) * p->gamma_q16) >> 16;"),
    ("eq4 sign", "const int64_t B = p->ttft_ns[cls[r]] - L;", "const int64_t B = p->ttft_ns[cls[r]] + L;"),
    ("eq5 sign", "const int64_t B_rem = B - elapsed;", "const int64_t B_rem = B + elapsed;"),
    ("tier test", "const int tier = (B > 0) ? 1 : 2;", "const int tier = (B >= 0) ? 1 : 2;"),
    ("attention term sign", "p->c_attn_q20 * (P * P - s * s)", "p->c_attn_q20 * (P * P + s * s)"),
    ("eq6 overhead charged for nothing", "return x == 0 ? 0 : p->delta_ns[k] + x * p->blk_ns[k];",
     "return p->delta_ns[k] + x * p->blk_ns[k];"),
    ("eq7 rounds up", "return std::min<int64_t>(nk, head / p->blk_ns[k]);",
     "return std::min<int64_t>(nk, (head + p->blk_ns[k] - 1) / p->blk_ns[k]);"),
    ("key shift", "(uint64_t(u) << 23)", "(uint64_t(u) << 24)"),
    ("maximum-load regime off by one", "std::max<int64_t>(D_act, p->max_batch - 1)",
     "std::max<int64_t>(D_act, p->max_batch)"),
    ("decode step without the request itself", "const Load act1{act.D + 1, act.K + P};",
     "const Load act1{act.D, act.K + P};"),
    ("penalty ignores the class target", "pen = O * std::max<int64_t>(0, tdec - tpot);",
     "pen = O * std::max<int64_t>(0, tdec);"),
    ("reserve not limited by tier-2 demand",
     "const int64_t R2 = std::min<int64_t>(std::min<int64_t>(p->tier2_reserve, W2), TB);",
     "const int64_t R2 = std::min<int64_t>(p->tier2_reserve, TB);"),
    ("decodes do not take tokens", "std::max<int64_t>(0, int64_t(p->token_budget) - D_act)",
     "std::max<int64_t>(0, int64_t(p->token_budget))"),
    ("batch cap off by one", "if (rank >= seq_cap) grant_out[r] = 0;", "if (rank > seq_cap) grant_out[r] = 0;"),
    ("tie goes to recompute", "if (F <= bF) { bF = F; bx1 = x1max; bx2 = 0; }",
     "if (F < bF) { bF = F; bx1 = x1max; bx2 = 0; }"),
    ("deep fetch still runs tokens", "const int64_t run = (bx2 > 0) ? 0 : std::min<int64_t>(grant[r], P - have);",
     "const int64_t run = std::min<int64_t>(grant[r], P - have);"),
    ("capacity cut off by one", "if (c > cap) {", "if (c >= cap) {"),
    ("victims walked from the front", "for (int i = n - 1; i >= 0; --i) {", "for (int i = 0; i < n; ++i) {"),
    ("shared holders preempted",
     "const bool eligible = valid[r] && grant[r] <= 0 && (flags[r] & ORC_FLAG_HBM_PRIVATE) && n0[r] > 0;",
     "const bool eligible = valid[r] && grant[r] <= 0 && n0[r] > 0;"),
    ("host room test off by one", "if (fits && h + n0[r] <= host_cnt)", "if (fits && h + n0[r] < host_cnt)"),
    ("evict list swapped", "evict_src[n_evict] = g; evict_dst[n_evict] = hslot;",
     "evict_src[n_evict] = hslot; evict_dst[n_evict] = g;"),
    ("restore reads the wrong table column", "restore_src[n_restore] = host_tbl[int64_t(r) * maxb + j];",
     "restore_src[n_restore] = host_tbl[int64_t(r) * maxb + j - n0[r]];"),
    ("record chunks strided like the pool", "host_pool + s * bb + c * chunk_bytes", "host_pool + s * bb + c * chunk_stride"),
    ("evict copies the wrong way", "std::memcpy(host_pool + d * bb + c * chunk_bytes, hbm_pool + c * chunk_stride + s * block_stride,",
     "std::memcpy(const_cast<uint8_t *>(hbm_pool) + c * chunk_stride + s * block_stride, host_pool + d * bb + c * chunk_bytes,"),
    ("prefetch ignores the admitted set's link time", "if (ok && grant[r] > 0) link_left -= restore_time(p, 1, x1[r]);",
     "if (ok && grant[r] > 0) link_left -= 0;"),
    ("prefetch serves preempted requests", "if (action[r] == ORC_ACT_EVICT || action[r] == ORC_ACT_DROP) continue;", ""),
    ("edf uses the wrong sign", "v = p->ttft_ns[cls[r]] - elapsed; tier2 = false;", "v = p->ttft_ns[cls[r]] + elapsed; tier2 = false;"),
    ("plan-first offer ignores the restore choice", "want[r] = x2 > 0 ? 0 : int64_t(prompt[r]) - (n0[r] + x1) * p->bt;",
     "want[r] = x2 > 0 ? 0 : int64_t(prompt[r]) - (n0[r] + n1[r]) * p->bt;"),
    ("plan-first offer for a staged deep fetch", "want[r] = x2 > 0 ? 0 : int64_t(prompt[r]) - (n0[r] + x1) * p->bt;",
     "want[r] = int64_t(prompt[r]) - (n0[r] + x1) * p->bt;"),
    ("regime 1 reuses the prefix", "lat4_out[4 * r + 1] = comp_q(p, tok_q(p, act), P, 0) >> 20;",
     "lat4_out[4 * r + 1] = comp_q(p, tok_q(p, act), P, s_hit) >> 20;"),
    # second batch: boundaries and terms the first batch did not touch
    ("class index test off by one", "ok = ok && cls[r] < p->n_classes;", "ok = ok && cls[r] <= p->n_classes;"),
    ("predicted output bound ignored", "ok = ok && O >= 0 && O <= (int64_t(1) << 20);", "ok = ok && O >= 0;"),
    ("transfer of the deep part left out of the estimate",
     "const int64_t tp = restore_time(p, 1, n1[r]) + restore_time(p, 2, n2[r]);\n        const int64_t L_act",
     "const int64_t tp = restore_time(p, 1, n1[r]);\n        const int64_t L_act"),
    ("maximum-load estimate uses the actual load",
     "const int64_t L_max = tp + (comp_q(p, tok_q(p, mx), P, s_hit) >> 20);\n        /* B3",
     "const int64_t L_max = tp + (comp_q(p, tok_q(p, act), P, s_hit) >> 20);\n        /* B3"),
    ("decode step leaves out the prefill chunk", "const int64_t tdec_act = (iter_q(p, act1) + chunk_q) >> 20;",
     "const int64_t tdec_act = (iter_q(p, act1)) >> 20;"),
    ("clamp one too wide", "std::min(std::max(v, -kBudgetClamp), kBudgetClamp - 1) + kBudgetClamp;",
     "std::min(std::max(v, -kBudgetClamp), kBudgetClamp) + kBudgetClamp;"),
    ("fcfs newest first", "if (p->policy == ORC_POLICY_FCFS) { v = -elapsed; tier2 = false; }",
     "if (p->policy == ORC_POLICY_FCFS) { v = elapsed; tier2 = false; }"),
    ("sjf by whole prompt", "if (p->policy == ORC_POLICY_SJF) { v = P - s_hit; tier2 = false; }",
     "if (p->policy == ORC_POLICY_SJF) { v = P; tier2 = false; }"),
    ("sort not stable", "std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return key[a] < key[b]; });",
     "std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return key[a] < key[b] || (key[a] == key[b] && a > b); });"),
    ("offer ignores the deep part", "want[r] = int64_t(prompt[r]) - int64_t(n0[r] + n1[r] + n2[r]) * p->bt;",
     "want[r] = int64_t(prompt[r]) - int64_t(n0[r] + n1[r]) * p->bt;"),
    ("tier-2 queue does not get what tier-1 left", "left = TB - used1;", "left = R2;"),
    ("regime 0 under the actual load", "lat4_out[4 * r + 0] = comp_q(p, tok_q(p, idle), P, 0) >> 20;",
     "lat4_out[4 * r + 0] = comp_q(p, tok_q(p, act), P, 0) >> 20;"),
    ("deep bound forgets the host transfer", "const int64_t rem2 = rem - restore_time(p, 1, n1);", "const int64_t rem2 = rem;"),
    ("need forgets the partly filled block", "need[r] = int32_t(bx1 + (ceil_div(have + run, p->bt) - (n0[r] + bx1)));",
     "need[r] = int32_t(bx1 + ((have + run) / p->bt - (n0[r] + bx1)));"),
    ("spill test ignores the victim's budget", "const bool fits = restore_time(p, 1, n0[r]) <= budget[r];",
     "const bool fits = true;"),
    ("deficit off by one", "const int64_t deficit = std::max<int64_t>(0, need_total - hbm_cnt);",
     "const int64_t deficit = std::max<int64_t>(0, need_total - hbm_cnt + 1);"),
    ("prefetch bound ignores the reserve", "int64_t avail = hbm_pos - hbm_reserve;", "int64_t avail = hbm_pos;"),
    ("prefetch restores although recomputing is cheaper",
     "if (m > 0 && plan_cost_q20(p, act, prompt[r], n0[r], m, 0) > plan_cost_q20(p, act, prompt[r], n0[r], 0, 0)) m = 0;", ""),
    ("prefetch link test forgets the overhead",
     "const int64_t by_link = link_left > p->delta_ns[1] ? (link_left - p->delta_ns[1]) / p->blk_ns[1] : 0;",
     "const int64_t by_link = link_left / p->blk_ns[1];"),
    # third batch
    ("host room counted for victims that are dropped anyway", "if (fits) h += n0[r];", "h += n0[r];"),
    ("one victim too many", "if (v < deficit) {", "if (v <= deficit) {"),
    ("evicted block recorded one cell off", "host_tbl[int64_t(r) * maxb + j] = hslot;", "host_tbl[int64_t(r) * maxb + j + 1] = hslot;"),
    ("admitted holders counted as preemptable",
     "if (valid[r] && grant[r] <= 0 && (flags[r] & ORC_FLAG_HBM_PRIVATE)) evictable += n0[r];",
     "if (valid[r] && (flags[r] & ORC_FLAG_HBM_PRIVATE)) evictable += n0[r];"),
    ("restored blocks not counted as held", "const int64_t have = (n0[r] + bx1) * int64_t(p->bt);",
     "const int64_t have = (n0[r]) * int64_t(p->bt);"),
    ("runs one token past the prompt", "const int64_t run = (bx2 > 0) ? 0 : std::min<int64_t>(grant[r], P - have);",
     "const int64_t run = (bx2 > 0) ? 0 : std::min<int64_t>(grant[r], P - have + 1);"),
    ("tier-1 count from the wrong bit", "if (key[r] >> 63)\n            W2 += want[r];", "if (key[r] >> 62)\n            W2 += want[r];"),
    ("unadmitted request keeps its restore", "x1_out[r] = x2_out[r] = tokens_run_out[r] = 0;\n            need[r] = 0;",
     "x2_out[r] = tokens_run_out[r] = 0;\n            need[r] = 0;"),
    ("victim keeps its table row", "if (with_tables) hbm_tbl[int64_t(r) * maxb + j] = -1;", ""),
    ("retain mark for requests without blocks", "if (valid[r] && action_out[r] == ORC_ACT_NONE && n0[r] > 0) action_out[r] = ORC_ACT_RETAIN;",
     "if (valid[r] && action_out[r] == ORC_ACT_NONE) action_out[r] = ORC_ACT_RETAIN;"),
    ("copy skips the last chunk", "for (int c = 0; c < n_chunks; ++c)\n            std::memcpy(hbm_pool + c * chunk_stride + d * block_stride,",
     "for (int c = 0; c + 1 < n_chunks; ++c)\n            std::memcpy(hbm_pool + c * chunk_stride + d * block_stride,"),
    # the deep-tier stage, the one-copy-per-source pass and the record copy have pins of their own
    ("stage hop charged the whole path", "std::max<int64_t>(0, p->delta_ns[2] - p->delta_ns[1]);",
     "std::max<int64_t>(0, p->delta_ns[2]);", DEEP_PINS),
    ("stage hop per block charged the whole path", "std::max<int64_t>(1, p->blk_ns[2] - p->blk_ns[1]);",
     "std::max<int64_t>(1, p->blk_ns[2]);", DEEP_PINS),
    ("stage ignores the host reserve", "int64_t room = host_pos - host_reserve;", "int64_t room = host_pos;", DEEP_PINS),
    ("stage writes the host segment's cells", "const int64_t t = int64_t(r) * maxb + n0[r] + n1[r] + j;",
     "const int64_t t = int64_t(r) * maxb + n0[r] + j;", DEEP_PINS),
    ("stage list swapped", "stage_src[n_stage] = deep_tbl[t]; stage_dst[n_stage] = rec;",
     "stage_src[n_stage] = rec; stage_dst[n_stage] = deep_tbl[t];", DEEP_PINS),
    ("stage serves preempted requests", "if (preempted) continue;", "", DEEP_PINS),
    ("stage forgets the per-transfer overhead", "link_left -= hop_delta + b * hop_blk;", "link_left -= b * hop_blk;",
     DEEP_PINS),
    ("stage takes the deep fetch although the host segment is cut", "if (bx2 <= 0) continue;",
     "bx2 = std::max<int64_t>(bx2, bx1 < n1[r] ? 1 : bx2); if (bx2 <= 0) continue;", DEEP_PINS),
    ("merged copy frees the kept block", "if (fpos < free_cap) free_list[fpos] = d; else status |= ORC_ST_EBOUNDS;",
     "if (fpos < free_cap) free_list[fpos] = kept[s]; else status |= ORC_ST_EBOUNDS;", DEEP_PINS),
    ("share count off by one", "ref[kept[s]] = merged[s];", "ref[kept[s]] = merged[s] - 1;", DEEP_PINS),
    ("every merged cell counts as shared", "if (merged[s] > 1) shared = 1;", "if (merged[s] >= 1) shared = 1;", DEEP_PINS),
    ("merged cells keep their own block", "dst_tbl[int64_t(r) * maxb + j] = kept[s];", "", DEEP_PINS),
    ("record copy the wrong way", "std::memcpy(host_pool + d * block_bytes, deep_pool + s * block_bytes, size_t(block_bytes));",
     "std::memcpy(host_pool + s * block_bytes, deep_pool + d * block_bytes, size_t(block_bytes));", DEEP_PINS),
]


def run_pins(env, pins=None):
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider"] + [os.path.join(ROOT, "tests", f) for f in pins or PINS]
    return subprocess.run(cmd, env=env, cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)


def test_every_planted_slip_is_caught(tmp_path):
    from concurrent.futures import ThreadPoolExecutor
    text = open(SRC).read()

    def survives(item):
        i, (name, old, new, *pins) = item
        assert text.count(old) == 1, f"mutation '{name}' no longer matches the source exactly once"
        path = tmp_path / f"mutant_{i}.cpp"
        path.write_text(text.replace(old, new))
        env = dict(os.environ, CASCADE_ORACLE_SRC=str(path))
        return name if run_pins(env, pins[0] if pins else None).returncode == 0 else None

    with ThreadPoolExecutor(max_workers=max(1, min(8, (os.cpu_count() or 2) // 2))) as pool:
        survivors = [s for s in pool.map(survives, enumerate(MUTATIONS)) if s]
    assert not survivors, f"pins did not notice: {survivors}"


def test_the_unaltered_copy_passes(tmp_path):
    path = tmp_path / "copy.cpp"
    path.write_text(open(SRC).read())
    res = run_pins(dict(os.environ, CASCADE_ORACLE_SRC=str(path)), PINS + DEEP_PINS)
    assert res.returncode == 0, res.stdout[-2000:]


def test_pins_pass_under_the_undefined_behaviour_sanitizer(tmp_path):
    """Signed overflow, bad shifts and out-of-range indexing in the oracle would make its outputs meaningless:
    the whole pin suite is run once more on a copy built with -fsanitize=undefined (any report aborts)."""
    path = tmp_path / "ubsan.cpp"
    path.write_text(open(SRC).read())
    env = dict(os.environ, CASCADE_ORACLE_SRC=str(path),
               CASCADE_ORACLE_CXXFLAGS="-fsanitize=undefined -fno-sanitize-recover=all -g")
    res = run_pins(env, PINS + DEEP_PINS)
    assert res.returncode == 0, res.stdout[-3000:]
