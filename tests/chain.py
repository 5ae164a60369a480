"""Shared test plumbing: the whole plan chain (plan, prefetch, merge, stage, merge) on the CPU oracle."""
import numpy as np

import oracle
from helpers import oracle_iteration


def oracle_chain(w, link, hbm_reserve, stage_link, host_reserve):
    res = oracle_iteration(w)
    plan, pools, r = res["plan"], res["pools"], w.reqs
    p = oracle.make_params(w.params)
    pf = oracle.prefetch_plan(p, r, res["budget"], res["order"], res["grant"], plan["action"], plan["x1"], w.D_act,
                              w.K_act, link, hbm_reserve, pools, plan["restore_src"], plan["restore_dst"])
    hbm_ref = np.zeros(w.layout["n_blocks"], np.int32)
    host_ref = np.zeros(w.host_blocks, np.int32)
    dr = oracle.dedup(r["n0"], None, plan["x1"], pf["pf"], pools.host_tbl, pools.hbm_tbl, pf["restore_src"],
                      pf["restore_dst"], len(pf["restore_src"]), w.host_blocks, w.layout["n_blocks"], pools.hbm_free,
                      pools.hbm_free_count, hbm_ref)
    pools.hbm_free_count = dr["free_count"]
    st = oracle.stage_plan(p, r, res["budget"], res["order"], plan["action"], w.D_act, w.K_act, stage_link,
                           host_reserve, pools, w.deep_tbl, len(w.host_free))
    ds = oracle.dedup(r["n0"], r["n1"], st["staged"], None, w.deep_tbl, pools.host_tbl, st["stage_src"],
                      st["stage_dst"], len(st["stage_src"]), w.deep_blocks, w.host_blocks, pools.host_free,
                      pools.host_free_count, host_ref)
    pools.host_free_count = ds["free_count"]
    return dict(res=res, pf=pf, dr=dr, st=st, ds=ds, hbm_ref=hbm_ref, host_ref=host_ref)
