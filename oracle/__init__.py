"""Plain CPU oracle for the BiLD decode loop.  TEST INFRASTRUCTURE ONLY: used by
tests/, the smoke check and the benchmark's CPU-baseline leg; never by the
product path, with which it shares no code."""
