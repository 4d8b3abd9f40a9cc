"""The library's self-tests: per-device bookkeeping of the launch sites (host only) and the bounded
device-side wait that backs PSKV_ERR_DEVICE_TIMEOUT (a tiny kernel whose wait runs out; no production
kernel is made to time out, and nothing faults or hangs)."""
import numpy as np
import pytest
import torch

import paper_2603_13420_b200 as pskv
from paper_2603_13420_b200.inputs import WORKLOADS

import parity


def test_per_device_guard_table_keeps_devices_apart():
    # two made-up device ordinals: marking one must not mark the other
    assert pskv.pskv_selftest_per_device_once() == 0


def test_multi_form_setter_rejects_unknown_values():
    with pytest.raises(pskv.PskvError):
        pskv.pskv_set_multi_form(7)
    pskv.pskv_set_multi_form("passes")
    pskv.pskv_set_multi_form("auto")


@pytest.mark.gpu
def test_a_wait_that_runs_out_reports_device_timeout_once_and_leaves_the_device_usable():
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    pskv.pskv_selftest_wait_timeout(100000)   # about 50 microseconds of waiting for a barrier nobody completes
    assert pskv.pskv_poll_device_status() == pskv.PSKV_ERR_DEVICE_TIMEOUT
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK   # reading the word clears it
    # the context is intact: an ordinary forward call still matches the oracle
    parity.fwd_parity(WORKLOADS["C0"], strict_abs=False)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK


@pytest.mark.gpu
def test_selftest_rejects_budgets_outside_its_range():
    with pytest.raises(pskv.PskvError):
        pskv.pskv_selftest_wait_timeout(0)
    with pytest.raises(pskv.PskvError):
        pskv.pskv_selftest_wait_timeout(10 ** 10)
