"""Seeded synthetic inputs (``workload``) and the device-side holder of a case (``device_case``) shared by
the tests, ``bench.py`` and the smoke check.  Neither holds any of the method's arithmetic; neither is
part of the library."""
