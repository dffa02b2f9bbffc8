"""Native measuring aids of the benchmark (bandwidth probe, C switch loop); not part of the library."""
